// Streaming norm-test kernel (optionally fused with AdamW) and its finalize kernel.
//
// Work decomposition.  Each shard of the flat vector is cut into chunks of
// `chunk_elems` consecutive coordinates (the last chunk of a shard may be short; a
// chunk never straddles a shard boundary).  A CTA processes whole chunks.  Inside a
// chunk, row r assigns the V = 16/sizeof(grad) consecutive coordinates starting at
// chunk_lo + (r*kThreads + tid)*V to thread tid, so the coordinate -> thread -> partial
// sum mapping depends only on (shard offsets, chunk_elems), never on the grid.  One
// record per chunk goes to scratch -- {n2, S, Q} (Q only in the diagnostic mode, else NaN), or
// {n2, S, index, ratio} of the chunk's largest per-coordinate ratio in the coordinate-wise
// mode; the finalize kernel combines chunk records in a fixed order per shard and shard
// records in shard order.
//
// Per coordinate (Algorithm 1, "Compute the batch gradient" .. "approximate gradient
// variance"): gbar = fp32(sum_k g_k / K).  fp32 inputs are summed in fp64, so gbar is the
// correctly rounded mean even under heavy cancellation.  bf16 inputs are summed in fp32,
// k = 0..K-1 in order: every partial sum is exact unless the addends' exponents spread
// over more than 13 binades (8-bit significands in a 24-bit accumulator), and fp64
// conversions would cost ~3% of bandwidth at the power cap.  Deviations g_k - gbar and
// their squares (and, in the diagnostic mode, g_k^2) are fp32 over at most V*K terms per
// thread-row, then accumulated in fp64.  The fused kernels and the many-worker kernel do
// this arithmetic two adjacent coordinates at a time with the packed fp32 instructions of
// sm_100 (coord_math_pair, adamw_pair); every lane rounds like the scalar instruction, so
// packed and scalar code give the same bits.
#pragma once
#include <cooperative_groups.h>

#include <type_traits>

#include "abs_device.cuh"

namespace absnt {

// What a kernel accumulates besides gbar: the two sums of the test always; the diagnostic
// Q = sum_k ||g_k||^2 on request; or, for the coordinate-wise test (Sec. 4, Proposition 1),
// the largest per-coordinate ratio sum_k (g_k[i]-gbar_i)^2 / gbar_i^2 and where it occurs.
// kStatNone: no statistics at all (the stand-alone AdamW update runs as the one-worker fused
// kernel in this mode: nothing is reduced, no chunk record is written).
enum StatMode { kStatSums = 0, kStatSumsQ = 1, kStatCoordwise = 2, kStatNone = 3 };

// Running maximum of the per-coordinate ratio within one thread, then one chunk.  The ratio is
// formed in fp32 with the hardware reciprocal (2^-22 relative).  A coordinate with zero
// deviations and zero mean gives 0 * inf = NaN, one with a non-finite input gives NaN as well:
// NaN never compares greater, so such coordinates are skipped here (non-finite inputs are
// reported through the sums).  Zero mean with positive deviations gives +inf.  Ties keep the
// lower index: a thread visits its coordinates in increasing order and replaces only on a
// strictly greater ratio.
struct CwMax {
  float r;
  int idx;  // coordinate index relative to the chunk's first coordinate
  __device__ __forceinline__ void init(int first_idx) {
    r = 0.f;
    idx = first_idx;
  }
  __device__ __forceinline__ void update(float dev2, float mean, int i) {
    float inv;
    asm("rcp.approx.f32 %0, %1;" : "=f"(inv) : "f"(mean * mean));
    const float q = dev2 * inv;
    if (q > r) {
      r = q;
      idx = i;
    }
  }
  __device__ __forceinline__ void merge(float r2, int idx2) {
    if (r2 > r || (r2 == r && idx2 < idx)) {
      r = r2;
      idx = idx2;
    }
  }
};

// Mean, squared deviations and (optionally) squared values of one coordinate.
template <typename GT, int KB, bool EXACT, bool WITHQ>
__device__ __forceinline__ float coord_math(const float (&g)[KB], int K, const StreamParams& prm,
                                            float& dev2, float& sq) {
  constexpr bool POW2 = EXACT && ((KB & (KB - 1)) == 0);
  typename GT::sum_t s = 0;
#pragma unroll
  for (int k = 0; k < KB; ++k)
    if (EXACT || k < K) s += static_cast<typename GT::sum_t>(g[k]);
  const float mean = GT::template mean<POW2>(s, prm);
  dev2 = 0.f;
  sq = 0.f;
#pragma unroll
  for (int k = 0; k < KB; ++k)
    if (EXACT || k < K) {
      const float dv = g[k] - mean;
      dev2 = fmaf(dv, dv, dev2);
      if (WITHQ) sq = fmaf(g[k], g[k], sq);
    }
  return mean;
}

// coord_math for two adjacent coordinates at once (lane x = the lower coordinate) with the
// packed fp32 instructions of sm_100.  Each lane performs the operations of coord_math in
// the same order with the same roundings, so the results are bit-identical to it.
template <typename GT, int KB, bool EXACT, bool WITHQ>
__device__ __forceinline__ float2 coord_math_pair(const float2 (&g)[KB], int K,
                                                  const StreamParams& prm, float2& dev2,
                                                  float2& sq) {
  constexpr bool POW2 = EXACT && ((KB & (KB - 1)) == 0);
  float2 mean;
  if constexpr (std::is_same<typename GT::sum_t, float>::value) {
    float2 s = make_float2(0.f, 0.f);
#pragma unroll
    for (int k = 0; k < KB; ++k)
      if (EXACT || k < K) s = __fadd2_rn(s, g[k]);
    mean = mean_of_sum2<POW2>(s, prm.inv_Kf, prm.neg_Kf);
  } else {
    typename GT::sum_t sx = 0, sy = 0;
#pragma unroll
    for (int k = 0; k < KB; ++k)
      if (EXACT || k < K) {
        sx += static_cast<typename GT::sum_t>(g[k].x);
        sy += static_cast<typename GT::sum_t>(g[k].y);
      }
    mean = make_float2(GT::template mean<POW2>(sx, prm), GT::template mean<POW2>(sy, prm));
  }
  const float2 neg_mean = make_float2(-mean.x, -mean.y);
  dev2 = make_float2(0.f, 0.f);
  sq = make_float2(0.f, 0.f);
#pragma unroll
  for (int k = 0; k < KB; ++k)
    if (EXACT || k < K) {
      const float2 dv = __fadd2_rn(g[k], neg_mean);
      dev2 = __ffma2_rn(dv, dv, dev2);
      if (WITHQ) sq = __ffma2_rn(g[k], g[k], sq);
    }
  return mean;
}

// Workers per group of the many-worker kernel: the loads of one group are issued together, and
// the shifted squares are accumulated per group and the group totals added up.  A flat fp32
// accumulation over hundreds of workers is biased for bf16 inputs (their squares are short bit
// patterns that hit rounding ties: S came out 1.4e-6 low at K = 333, 2.5e-6 low at K = 1024);
// with group totals the error is 3e-8 at K = 1024.  Compile-time worker counts use 16; the
// run-time loop 16 for bf16 (8-byte vectors) and 8 for fp32.
template <typename GT, bool EXACT>
__host__ __device__ constexpr int split_group() {
  return EXACT ? 16 : (sizeof(typename GT::raw_t) <= 8 ? 16 : 8);
}

// The same three quantities with the shifted one-pass form used for many workers:
//   c = g_0;  S_i = sum_k (g_k - c)^2 - K (gbar - c)^2
// so that the K values need not all be live at once.  The cancellation is bounded: the
// first sum exceeds S_i by at most a factor of about K (when g_0 itself is the outlier).
// K identical values give exactly zero.
// The deviation of the mean, dm = gbar - c, is taken from the unrounded sum and not from the
// rounded mean: with s = sum_k g_k (exact in fp32 for bf16 inputs within the binade limits,
// fp64 for fp32 inputs), gbar = fl(s/K) as in the plain form, and dm = fl((s - K c)/K) -- for
// bf16 one fused multiply-add, whose exact result sum_k (g_k - c) is representable under the
// same limits; for fp32 one fp64 subtraction.  Were dm formed as fl(gbar) - c, the rounding
// error delta of gbar would enter S_i to first order (2 K dm delta: relative 2^-24 |mean| /
// spread, visible once the workers agree to four digits); this way it does not enter at all.
// The operation order is that of the vector path of chunk_rows_split, so both give identical
// bits.
template <typename GT, int KB, bool EXACT, bool WITHQ>
__device__ __forceinline__ float coord_math_split(const float (&g)[KB], int K,
                                                  const StreamParams& prm, float& dev2, float& sq) {
  constexpr bool kF32Sum = std::is_same<typename GT::sum_t, float>::value;
  constexpr int H = split_group<GT, EXACT>();
  typename GT::sum_t s = 0;
  const float c = g[0];
  float s2 = 0.f, g2 = 0.f;  // total of the closed groups, the open group
  float gq = 0.f;            // the same for the plain squares
  sq = 0.f;
#pragma unroll
  for (int k = 0; k < KB; ++k)
    if (EXACT || k < K) {
      s += static_cast<typename GT::sum_t>(g[k]);
      const float dv = g[k] - c;
      g2 = fmaf(dv, dv, g2);
      if (WITHQ) gq = fmaf(g[k], g[k], gq);
      if ((k + 1) % H == 0 || k + 1 == (EXACT ? KB : K)) {
        s2 += g2;
        g2 = 0.f;
        if (WITHQ) {
          sq += gq;
          gq = 0.f;
        }
      }
    }
  float mean, dm;
  if constexpr (kF32Sum) {
    mean = mean_of_sum<false>(s, prm.inv_Kf, prm.neg_Kf);
    dm = fmaf(prm.neg_Kf, c, s) * prm.inv_Kf;
  } else {
    const double mx = s * prm.inv_K;
    mean = static_cast<float>(mx);
    dm = static_cast<float>(mx - static_cast<double>(c));
  }
  dev2 = clamp_nonneg(fmaf(prm.neg_Kf * dm, dm, s2));
  return mean;
}

// The V coordinates of one thread-row with element-wise, bounds-checked accesses: used for
// rows that are ragged (end of a shard) or whose streams are not 16-byte aligned.  Same
// arithmetic in the same order as the vector path, so both give identical bits.  Kept out
// of line so that its registers do not weigh on the vector path.
template <typename GT, int KB, bool EXACT, bool ADAM, int STAT, bool SPLIT = false>
__device__ __noinline__ void scalar_row(const StreamParams& prm, const void* const* grads, int K,
                                        int64_t base, int64_t hi, int64_t chunk_lo,
                                        float* sums /* n2, S, Q of this thread-row */,
                                        CwMax* cw, GradWeights gw) {
  constexpr int V = GT::kVec;
  constexpr bool WITHQ = STAT == kStatSumsQ;
  float row_n2 = 0.f, row_S = 0.f, row_Q = 0.f;
  for (int e = 0; e < V; ++e) {
    const int64_t i = base + e;
    if (i >= hi) break;  // the remaining coordinates would add exact zeros
    float dev2, sq, mean;
    if constexpr (SPLIT && !EXACT) {
      // any worker count: the arithmetic of coord_math_split with the values consumed as they
      // are loaded (same operations in the same order)
      constexpr bool kF32Sum = std::is_same<typename GT::sum_t, float>::value;
      constexpr int H = split_group<GT, false>();
      typename GT::sum_t s = 0;
      const float c = GT::load1(grads[0], i);
      float s2 = 0.f, g2 = 0.f, gq = 0.f;
      sq = 0.f;
      for (int k = 0; k < K; ++k) {
        const float g = GT::load1(grads[k], i);
        s += static_cast<typename GT::sum_t>(g);
        const float dv = g - c;
        g2 = fmaf(dv, dv, g2);
        if (WITHQ) gq = fmaf(g, g, gq);
        if ((k + 1) % H == 0 || k + 1 == K) {
          s2 += g2;
          g2 = 0.f;
          if (WITHQ) {
            sq += gq;
            gq = 0.f;
          }
        }
      }
      float dm;
      if constexpr (kF32Sum) {
        mean = mean_of_sum<false>(s, prm.inv_Kf, prm.neg_Kf);
        dm = fmaf(prm.neg_Kf, c, s) * prm.inv_Kf;
      } else {
        const double mx = s * prm.inv_K;
        mean = static_cast<float>(mx);
        dm = static_cast<float>(mx - static_cast<double>(c));
      }
      dev2 = clamp_nonneg(fmaf(prm.neg_Kf * dm, dm, s2));
    } else {
      float g[KB];
#pragma unroll
      for (int k = 0; k < KB; ++k) g[k] = (EXACT || k < K) ? GT::load1(grads[k], i) : 0.f;
      mean = SPLIT ? coord_math_split<GT, KB, EXACT, WITHQ>(g, K, prm, dev2, sq)
                   : coord_math<GT, KB, EXACT, WITHQ>(g, K, prm, dev2, sq);
    }
    row_n2 = fmaf(mean, mean, row_n2);
    row_S += dev2;
    row_Q += sq;
    if (STAT == kStatCoordwise) cw->update(dev2, mean, static_cast<int>(i - chunk_lo));
    if (prm.gbar) prm.gbar[i] = mean;
    if (ADAM) {
      float w = prm.p[i], m = prm.m[i], v = prm.v[i];
      adamw_elem(prm.adam, gw.omb1, gw.omb2, mean, w, m, v);
      prm.p[i] = w;
      prm.m[i] = m;
      prm.v[i] = v;
      if (prm.p16) prm.p16[i] = to_bf16(w);
    }
  }
  sums[0] = row_n2;
  sums[1] = row_S;
  sums[2] = row_Q;
}

// Where a chunk lies and how its streams are aligned (uniform across the CTA; computed
// from kernel parameters only).
struct ChunkGeometry {
  int64_t lo, hi;  // coordinates [lo, hi)
  bool aligned;    // every stream 16-byte aligned at lo: vector path
  bool wide;       // fp32 arrays also 32-byte aligned: 256-bit accesses (bf16 gradients)
};

template <typename GT, int KB, bool EXACT, bool ADAM>
__device__ __forceinline__ ChunkGeometry chunk_geometry(const StreamParams& prm,
                                                        const void* const* grads, int K,
                                                        int chunk) {
  // shard that owns this chunk: largest s with chunk_prefix[s] <= chunk
  int lo_s = 0, hi_s = prm.n_shards;
  while (hi_s - lo_s > 1) {
    const int mid = (lo_s + hi_s) >> 1;
    if (prm.chunk_prefix[mid] <= chunk) lo_s = mid; else hi_s = mid;
  }
  ChunkGeometry g;
  g.lo = prm.shard_off[lo_s] +
         static_cast<int64_t>(chunk - prm.chunk_prefix[lo_s]) * prm.chunk_elems;
  const int64_t shard_hi = prm.shard_off[lo_s + 1];
  g.hi = (g.lo + prm.chunk_elems < shard_hi) ? g.lo + prm.chunk_elems : shard_hi;
  uintptr_t bits = 0, bits_f32 = 0;
  if constexpr (EXACT) {
#pragma unroll
    for (int k = 0; k < KB; ++k)
      bits |= reinterpret_cast<uintptr_t>(grads[k]) +
              static_cast<uintptr_t>(g.lo) * sizeof(typename GT::scalar);
  } else {
    for (int k = 0; k < K; ++k)
      bits |= reinterpret_cast<uintptr_t>(grads[k]) +
              static_cast<uintptr_t>(g.lo) * sizeof(typename GT::scalar);
  }
  if (prm.gbar) bits_f32 |= reinterpret_cast<uintptr_t>(prm.gbar) + static_cast<uintptr_t>(g.lo) * 4;
  if (ADAM) {
    bits_f32 |= reinterpret_cast<uintptr_t>(prm.p) + static_cast<uintptr_t>(g.lo) * 4;
    bits_f32 |= reinterpret_cast<uintptr_t>(prm.m) + static_cast<uintptr_t>(g.lo) * 4;
    bits_f32 |= reinterpret_cast<uintptr_t>(prm.v) + static_cast<uintptr_t>(g.lo) * 4;
    if (prm.p16) bits |= reinterpret_cast<uintptr_t>(prm.p16) + static_cast<uintptr_t>(g.lo) * 2;
  }
  g.aligned = ((bits | bits_f32) & 15) == 0;
  g.wide = (GT::kVec == 8) && (bits_f32 & 31) == 0;
  return g;
}

// Register-direct processing of one chunk: every thread-row is loaded with 128/256-bit
// global loads straight into registers.  Adds this thread's sums to acc_*.
template <typename GT, int KB, bool EXACT, bool ADAM, int STAT, int NT = kThreads>
__device__ __forceinline__ void chunk_rows_direct(const StreamParams& prm, int K,
                                                  const ChunkGeometry& cg, double& acc_n2,
                                                  double& acc_S, double& acc_Q, CwMax& cw,
                                                  GradWeights gw) {
  constexpr int V = GT::kVec;
  constexpr bool WITHQ = STAT == kStatSumsQ;
  constexpr bool CW = STAT == kStatCoordwise;
  constexpr int NF4 = V / 4; // float4 per thread-row of an fp32 array
  // 256-bit stores of the fp32 arrays pay off for few workers (K <= 7: +3..9% measured) and
  // cost about 1% for K >= 8, where the stores of the first half are better issued early;
  // 256-bit loads never hurt.
  constexpr bool kWideStores = (V == 8) && (KB < 8 || !EXACT) && KB <= 8;
  const int tid = threadIdx.x;
  const int64_t hi = cg.hi;
  const bool wide = cg.wide;
  int64_t row_lo = cg.lo;

  // The test alone moves few bytes per coordinate (K*s + 4), so with few workers one thread-row
  // of K vectors leaves too little in flight (K=4 bf16: 49 KB per SM, 68% DRAM utilisation,
  // warps stalled on loads).  For K <= 4, while full aligned rows remain, 8/K of them are
  // loaded before the first is consumed (eight vectors per thread, still three CTAs per SM);
  // the rows are consumed in order, so the sums keep their shape.  Measured at d = 124M, bf16 /
  // fp32: K=1 5.7 -> 6.4 / 5.1 -> 6.2 TB/s, K=2 5.9 -> 6.5 / 5.5 -> 6.5, K=4 5.9 -> 6.6 / 6.3 ->
  // 6.5.  Sixteen vectors per thread at two CTAs per SM lose for bf16 (K=8: 6.6 -> 6.2).
  constexpr int kRows = (!ADAM && EXACT && KB <= 4) ? 8 / KB : 1;
  if constexpr (kRows > 1) {
    while (cg.aligned && row_lo + static_cast<int64_t>(kRows) * NT * V <= hi) {
      typename GT::raw_t rawr[kRows][KB];
#pragma unroll
      for (int r = 0; r < kRows; ++r)
#pragma unroll
        for (int k = 0; k < KB; ++k)
          rawr[r][k] = GT::load_vec(reinterpret_cast<const typename GT::scalar*>(prm.grads[k]) +
                                    row_lo + static_cast<int64_t>(r) * NT * V +
                                    static_cast<int64_t>(tid) * V);
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        const int64_t base = row_lo + static_cast<int64_t>(r) * NT * V + static_cast<int64_t>(tid) * V;
        float row_n2 = 0.f, row_S = 0.f, row_Q = 0.f;
        float4 gbv[NF4];
#pragma unroll
        for (int q = 0; q < NF4; ++q) {
          float gb[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float g[KB];
#pragma unroll
            for (int k = 0; k < KB; ++k) g[k] = GT::elem(rawr[r][k], 4 * q + j);
            float dev2, sq;
            const float mean = coord_math<GT, KB, EXACT, WITHQ>(g, K, prm, dev2, sq);
            gb[j] = mean;
            row_n2 = fmaf(mean, mean, row_n2);
            row_S += dev2;
            row_Q += sq;
            if (CW) cw.update(dev2, mean, static_cast<int>(base - cg.lo) + 4 * q + j);
          }
          gbv[q] = make_float4(gb[0], gb[1], gb[2], gb[3]);
        }
        if (prm.gbar) {
          if (V == 8 && wide) {
            st_stream_32(prm.gbar + base, gbv[0], gbv[NF4 - 1]);
          } else {
#pragma unroll
            for (int q = 0; q < NF4; ++q) st_stream_16(prm.gbar + base + 4 * q, gbv[q]);
          }
        }
        acc_n2 += static_cast<double>(row_n2);
        acc_S += static_cast<double>(row_S);
        if (WITHQ) acc_Q += static_cast<double>(row_Q);
      }
      row_lo += static_cast<int64_t>(kRows) * NT * V;
    }
  }

  for (; row_lo < hi; row_lo += NT * V) {
    const int64_t base = row_lo + static_cast<int64_t>(tid) * V;
    float row_n2 = 0.f, row_S = 0.f, row_Q = 0.f;

    if (cg.aligned && (row_lo + NT * V <= hi)) {
      typename GT::raw_t raw[KB];
#pragma unroll
      for (int k = 0; k < KB; ++k)
        if (EXACT || k < K)
          raw[k] = GT::load_vec(reinterpret_cast<const typename GT::scalar*>(prm.grads[k]) + base);
      float4 pw[NF4], pm[NF4], pv[NF4];
      if (ADAM) {
        if (V == 8 && wide) {
          const Float8 a = ld_state_32(prm.p + base), b = ld_state_32(prm.m + base),
                       c = ld_state_32(prm.v + base);
          pw[0] = a.lo; pw[NF4 - 1] = a.hi;
          pm[0] = b.lo; pm[NF4 - 1] = b.hi;
          pv[0] = c.lo; pv[NF4 - 1] = c.hi;
        } else {
#pragma unroll
          for (int q = 0; q < NF4; ++q) {
            pw[q] = ld_state_16(prm.p + base + 4 * q);
            pm[q] = ld_state_16(prm.m + base + 4 * q);
            pv[q] = ld_state_16(prm.v + base + 4 * q);
          }
        }
      }
      // four coordinates at a time, stored as soon as they are done (short live ranges)
      float4 gb_lo = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int q = 0; q < NF4; ++q) {
        float gb[4];
        // Two coordinates per packed fp32 instruction in the fused kernels (+0.4..0.8% at
        // K = 16) and in the plain bf16 test with six workers (6.53 -> 6.62 TB/s; with eight it
        // costs 0.5%, and with Q computed the eight-vector kernels spill: bf16 K=2 6.5 -> 5.8
        // TB/s).  The row sums take the coordinates in index order, as scalar_row does.
        constexpr bool kPackedRow =
            ADAM || (STAT == kStatSums && EXACT && KB == 6 && GT::kVec == 8);
        if constexpr (kPackedRow) {
          float2* w2 = reinterpret_cast<float2*>(&pw[q]);
          float2* m2 = reinterpret_cast<float2*>(&pm[q]);
          float2* v2 = reinterpret_cast<float2*>(&pv[q]);
#pragma unroll
          for (int jp = 0; jp < 2; ++jp) {
            float2 g[KB];
#pragma unroll
            for (int k = 0; k < KB; ++k)
              g[k] = (EXACT || k < K) ? GT::pair(raw[k], 2 * q + jp) : make_float2(0.f, 0.f);
            float2 dev2, sq;
            const float2 mean = coord_math_pair<GT, KB, EXACT, WITHQ>(g, K, prm, dev2, sq);
            gb[2 * jp] = mean.x;
            gb[2 * jp + 1] = mean.y;
            row_n2 = fmaf(mean.x, mean.x, row_n2);
            row_n2 = fmaf(mean.y, mean.y, row_n2);
            row_S += dev2.x;
            row_S += dev2.y;
            row_Q += sq.x;
            row_Q += sq.y;
            if (CW) {
              const int li = static_cast<int>(base - cg.lo) + 4 * q + 2 * jp;
              cw.update(dev2.x, mean.x, li);
              cw.update(dev2.y, mean.y, li + 1);
            }
            if constexpr (ADAM) adamw_pair(prm.adam, gw.omb1, gw.omb2, mean, w2[jp], m2[jp], v2[jp]);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float g[KB];
#pragma unroll
            for (int k = 0; k < KB; ++k)
              g[k] = (EXACT || k < K) ? GT::elem(raw[k], 4 * q + j) : 0.f;
            float dev2, sq;
            const float mean = coord_math<GT, KB, EXACT, WITHQ>(g, K, prm, dev2, sq);
            gb[j] = mean;
            row_n2 = fmaf(mean, mean, row_n2);
            row_S += dev2;
            row_Q += sq;
            if (CW) cw.update(dev2, mean, static_cast<int>(base - cg.lo) + 4 * q + j);
          }
        }
        if (kWideStores && wide) {
          // hold the first half back; store all 32 bytes with the second half
          if (q == 0) {
            gb_lo = make_float4(gb[0], gb[1], gb[2], gb[3]);
          } else {
            if (prm.gbar)
              st_stream_32(prm.gbar + base, gb_lo, make_float4(gb[0], gb[1], gb[2], gb[3]));
            if (ADAM) {
              st_stream_32(prm.p + base, pw[0], pw[NF4 - 1]);
              st_stream_32(prm.m + base, pm[0], pm[NF4 - 1]);
              st_stream_32(prm.v + base, pv[0], pv[NF4 - 1]);
              if (prm.p16) st_bf16x8(prm.p16 + base, pw[0], pw[NF4 - 1]);
            }
          }
        } else {
          if (prm.gbar)
            st_stream_16(prm.gbar + base + 4 * q, make_float4(gb[0], gb[1], gb[2], gb[3]));
          if (ADAM) {
            st_stream_16(prm.p + base + 4 * q, pw[q]);
            st_stream_16(prm.m + base + 4 * q, pm[q]);
            st_stream_16(prm.v + base + 4 * q, pv[q]);
            if (prm.p16) st_bf16x4(prm.p16 + base + 4 * q, pw[q]);
          }
        }
      }
    } else if (base < hi) {
      float sums[3];
      scalar_row<GT, KB, EXACT, ADAM, STAT>(prm, prm.grads, K, base, hi, cg.lo, sums, &cw, gw);
      row_n2 = sums[0];
      row_S = sums[1];
      row_Q = sums[2];
    }
    acc_n2 += static_cast<double>(row_n2);
    acc_S += static_cast<double>(row_S);
    if (WITHQ) acc_Q += static_cast<double>(row_Q);
  }
}

// CTA-wide fixed-order reduction of the per-thread sums and the chunk record {n2, S, Q, 0}.
// Coordinate-wise mode: {n2, S, index of the chunk's largest ratio, that ratio}; the maximum
// is exact and order-independent, ties go to the lower index.
template <int STAT, int NT = kThreads>
__device__ __forceinline__ void write_chunk_record(const StreamParams& prm, int chunk,
                                                   int64_t chunk_lo, double acc_n2, double acc_S,
                                                   double acc_Q, CwMax cw, double* red) {
  if constexpr (STAT == kStatNone) return;
  constexpr bool WITHQ = STAT == kStatSumsQ;
  constexpr bool CW = STAT == kStatCoordwise;
  __shared__ float cw_r[NT / 32];
  __shared__ int cw_i[NT / 32];
  if (CW) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float r2 = __shfl_down_sync(0xffffffffu, cw.r, off);
      const int i2 = __shfl_down_sync(0xffffffffu, cw.idx, off);
      cw.merge(r2, i2);
    }
    if ((threadIdx.x & 31) == 0) {
      cw_r[threadIdx.x >> 5] = cw.r;
      cw_i[threadIdx.x >> 5] = cw.idx;
    }
  }
  block_reduce3<NT / 32>(acc_n2, acc_S, acc_Q, red);  // synchronises the CTA twice
  if (threadIdx.x == 0) {
    double* out = prm.chunk_out + static_cast<int64_t>(chunk) * 4;
    out[0] = acc_n2;
    out[1] = acc_S;
    if (CW) {
#pragma unroll
      for (int w = 1; w < NT / 32; ++w) cw.merge(cw_r[w], cw_i[w]);
      out[2] = static_cast<double>(chunk_lo + cw.idx);
      out[3] = static_cast<double>(cw.r);
    } else {
      out[2] = WITHQ ? acc_Q : __longlong_as_double(0x7ff8000000000000ll);  // NaN: not computed
      out[3] = 0.0;
    }
  }
  if (CW) __syncthreads();  // cw_r / cw_i are free again before a next chunk's warps write them
}

template <typename GT, int KB, bool EXACT, bool ADAM, int STAT>
__global__ void __launch_bounds__(kThreads, ((KB <= 8 && EXACT) ? 3 : ((KB <= 16 || GT::kVec * sizeof(typename GT::scalar) <= 8) ? 2 : 1)))
    normtest_stream_kernel(const __grid_constant__ StreamParams prm) {
  __shared__ double red[kWarps * 3];
  const int K = EXACT ? KB : prm.K;
  bool waited = false;
  GradWeights gw{prm.adam.omb1, prm.adam.omb2};
  for (int chunk = blockIdx.x; chunk < prm.n_chunks; chunk += gridDim.x) {
    const ChunkGeometry cg = chunk_geometry<GT, KB, EXACT, ADAM>(prm, prm.grads, K, chunk);
    if (!waited) {  // everything above used kernel parameters only
      grid_dependency_wait();
      waited = true;
      if (ADAM) gw = grad_weights(prm.adam, prm.clip_n2, prm.clip_max_norm);
    }
    double acc_n2 = 0.0, acc_S = 0.0, acc_Q = 0.0;
    CwMax cw;
    cw.init(static_cast<int>(threadIdx.x) * GT::kVec);
    chunk_rows_direct<GT, KB, EXACT, ADAM, STAT>(prm, K, cg, acc_n2, acc_S, acc_Q, cw, gw);
    write_chunk_record<STAT>(prm, chunk, cg.lo, acc_n2, acc_S, acc_Q, cw, red);
  }
}

// Register-direct processing for many workers, or for a worker count without an unrolled
// kernel of its own: the workers are taken in groups (two halves of 16 for K = 32; a
// run-time loop over groups of 8 otherwise) with the shifted one-pass form of
// coord_math_split, so only one group of gradient vectors is live per thread (two or three
// CTAs per SM instead of one at 255 registers, and no instructions for absent workers
// beyond the last group).
template <typename GT, int KB, bool EXACT, bool ADAM, int STAT>
__device__ __forceinline__ void chunk_rows_split(const StreamParams& prm,
                                                 const void* const* grads, int K,
                                                 const ChunkGeometry& cg, double& acc_n2,
                                                 double& acc_S, double& acc_Q, CwMax& cw,
                                                 GradWeights gw) {
  constexpr int V = GT::kVec;
  constexpr bool WITHQ = STAT == kStatSumsQ;
  constexpr bool CW = STAT == kStatCoordwise;
  static_assert(V == 4, "split path: four coordinates per thread-row");
  // exact K: compile-time groups of 16 and one group of K mod 16; any other K: a run-time loop
  // over groups of 32 bytes
  // per coordinate quad in registers (8 fp32 vectors, 16 bf16 vectors), then the remaining
  // workers in unpredicated pieces of 8, 4, 2 and 1
  constexpr int H = split_group<GT, EXACT>();
  static_assert(EXACT || KB % H == 0, "groups");
  const int tid = threadIdx.x;
  const int64_t hi = cg.hi;

  for (int64_t row_lo = cg.lo; row_lo < hi; row_lo += kThreads * V) {
    const int64_t base = row_lo + static_cast<int64_t>(tid) * V;
    float row_n2 = 0.f, row_S = 0.f, row_Q = 0.f;
    if (cg.aligned && (row_lo + kThreads * V <= hi)) {
      // two coordinates per packed fp32 instruction (pair p = coordinates 2p, 2p+1); each
      // lane does what coord_math_split does, in the same order
      constexpr bool kF32Sum = std::is_same<typename GT::sum_t, float>::value;
      constexpr int P = V / 2;
      typename GT::sum_t s[V];  // sums of fp32 gradients (fp64)
      float2 sp[P];             // sums of bf16 gradients (fp32, packed)
      float2 c[P], neg_c[P], s2[P], g2[P], q[P], gq[P];  // s2, q: closed groups; g2, gq: the open one
#pragma unroll
      for (int e = 0; e < V; ++e) s[e] = 0;
#pragma unroll
      for (int pi = 0; pi < P; ++pi)
        sp[pi] = c[pi] = neg_c[pi] = s2[pi] = g2[pi] = q[pi] = gq[pi] = make_float2(0.f, 0.f);
      auto close_group = [&]() {
#pragma unroll
        for (int pi = 0; pi < P; ++pi) {
          s2[pi] = __fadd2_rn(s2[pi], g2[pi]);
          g2[pi] = make_float2(0.f, 0.f);
          if (WITHQ) {
            q[pi] = __fadd2_rn(q[pi], gq[pi]);
            gq[pi] = make_float2(0.f, 0.f);
          }
        }
      };
      float4 pw, pm, pv;
      if (ADAM) {  // in flight while the gradients are consumed
        pw = ld_state_16(prm.p + base);
        pm = ld_state_16(prm.m + base);
        pv = ld_state_16(prm.v + base);
      }
      // N consecutive workers starting at k0, all present: loads first, then the arithmetic
      auto group = [&](int k0, auto n_tag) {
        constexpr int N = decltype(n_tag)::value;
        typename GT::raw_t raw[N];
#pragma unroll
        for (int k = 0; k < N; ++k)
          raw[k] = GT::load_vec(
              reinterpret_cast<const typename GT::scalar*>(grads[k0 + k]) + base);
#pragma unroll
        for (int pi = 0; pi < P; ++pi) {
#pragma unroll
          for (int k = 0; k < N; ++k) {
            const float2 g = GT::pair(raw[k], pi);
            if (k0 == 0 && k == 0) {
              c[pi] = g;
              neg_c[pi] = make_float2(-g.x, -g.y);
            }
            const float2 dv = __fadd2_rn(g, neg_c[pi]);
            if constexpr (kF32Sum) {
              sp[pi] = __fadd2_rn(sp[pi], g);
            } else {
              s[2 * pi] += static_cast<typename GT::sum_t>(g.x);
              s[2 * pi + 1] += static_cast<typename GT::sum_t>(g.y);
            }
            g2[pi] = __ffma2_rn(dv, dv, g2[pi]);
            if (WITHQ) gq[pi] = __ffma2_rn(g, g, gq[pi]);
          }
        }
      };
      if constexpr (EXACT) {
#pragma unroll
        for (int h = 0; h < KB / H; ++h) {
          group(h * H, std::integral_constant<int, H>{});
          close_group();
        }
        if constexpr (KB % H != 0) {
          group(KB / H * H, std::integral_constant<int, KB % H>{});
          close_group();
        }
      } else {
        // whole groups in a run-time loop, then the remainder in pieces of 8, 4, 2, 1 workers:
        // no load is predicated on the worker count
        int k0 = 0;
#pragma unroll 1
        for (; k0 + H <= K; k0 += H) {
          group(k0, std::integral_constant<int, H>{});
          close_group();
        }
        // the rest (fewer than H workers) is one more group, taken in pieces
        if (H > 8 && ((K - k0) & 8)) {
          group(k0, std::integral_constant<int, 8>{});
          k0 += 8;
        }
        if ((K - k0) & 4) {
          group(k0, std::integral_constant<int, 4>{});
          k0 += 4;
        }
        if ((K - k0) & 2) {
          group(k0, std::integral_constant<int, 2>{});
          k0 += 2;
        }
        if ((K - k0) & 1) group(k0, std::integral_constant<int, 1>{});
        close_group();  // adds exact zeros when K is a multiple of H
      }
      float gb[V];
      float2* w2 = reinterpret_cast<float2*>(&pw);
      float2* m2 = reinterpret_cast<float2*>(&pm);
      float2* v2 = reinterpret_cast<float2*>(&pv);
#pragma unroll
      for (int pi = 0; pi < P; ++pi) {
        float2 mean, dm;
        if constexpr (kF32Sum) {
          mean = mean_of_sum2<false>(sp[pi], prm.inv_Kf, prm.neg_Kf);
          dm = __fmul2_rn(__ffma2_rn(make_float2(prm.neg_Kf, prm.neg_Kf), c[pi], sp[pi]),
                          make_float2(prm.inv_Kf, prm.inv_Kf));
        } else {
          const double mx = s[2 * pi] * prm.inv_K, my = s[2 * pi + 1] * prm.inv_K;
          mean = make_float2(static_cast<float>(mx), static_cast<float>(my));
          dm = make_float2(static_cast<float>(mx - static_cast<double>(c[pi].x)),
                           static_cast<float>(my - static_cast<double>(c[pi].y)));
        }
        const float2 t = __ffma2_rn(__fmul2_rn(make_float2(prm.neg_Kf, prm.neg_Kf), dm), dm, s2[pi]);
        gb[2 * pi] = mean.x;
        gb[2 * pi + 1] = mean.y;
        row_n2 = fmaf(mean.x, mean.x, row_n2);
        row_n2 = fmaf(mean.y, mean.y, row_n2);
        const float tx = clamp_nonneg(t.x), ty = clamp_nonneg(t.y);
        row_S += tx;
        row_S += ty;
        row_Q += q[pi].x;
        row_Q += q[pi].y;
        if (CW) {
          const int li = static_cast<int>(base - cg.lo) + 2 * pi;
          cw.update(tx, mean.x, li);
          cw.update(ty, mean.y, li + 1);
        }
        if (ADAM) adamw_pair(prm.adam, gw.omb1, gw.omb2, mean, w2[pi], m2[pi], v2[pi]);
      }
      if (prm.gbar) st_stream_16(prm.gbar + base, make_float4(gb[0], gb[1], gb[2], gb[3]));
      if (ADAM) {
        st_stream_16(prm.p + base, pw);
        st_stream_16(prm.m + base, pm);
        st_stream_16(prm.v + base, pv);
        if (prm.p16) st_bf16x4(prm.p16 + base, pw);
      }
    } else if (base < hi) {
      float sums[3];
      scalar_row<GT, KB, EXACT, ADAM, STAT, true>(prm, grads, K, base, hi, cg.lo, sums, &cw, gw);
      row_n2 = sums[0];
      row_S = sums[1];
      row_Q = sums[2];
    }
    acc_n2 += static_cast<double>(row_n2);
    acc_S += static_cast<double>(row_S);
    if (WITHQ) acc_Q += static_cast<double>(row_Q);
  }
}

template <typename GT, int KB, bool EXACT, bool ADAM, int STAT>
__global__ void __launch_bounds__(kThreads, 2)
    normtest_split_kernel(const __grid_constant__ StreamParams prm) {
  __shared__ double red[kWarps * 3];
  const int K = EXACT ? KB : prm.K;
  bool waited = false;
  GradWeights gw{prm.adam.omb1, prm.adam.omb2};
  for (int chunk = blockIdx.x; chunk < prm.n_chunks; chunk += gridDim.x) {
    const ChunkGeometry cg = chunk_geometry<GT, KB, EXACT, ADAM>(prm, prm.grads, K, chunk);
    if (!waited) {
      grid_dependency_wait();
      waited = true;
      if (ADAM) gw = grad_weights(prm.adam, prm.clip_n2, prm.clip_max_norm);
    }
    double acc_n2 = 0.0, acc_S = 0.0, acc_Q = 0.0;
    CwMax cw;
    cw.init(static_cast<int>(threadIdx.x) * GT::kVec);
    chunk_rows_split<GT, KB, EXACT, ADAM, STAT>(prm, prm.grads, K, cg, acc_n2, acc_S, acc_Q, cw, gw);
    write_chunk_record<STAT>(prm, chunk, cg.lo, acc_n2, acc_S, acc_Q, cw, red);
  }
}

// Finalize: one thread-block cluster of 1, 2, 4 or 8 CTAs x kFinalizeThreads threads.
//
// Every shard's chunk records are cut into slices of fp.slice consecutive records (a power of
// two times 128, chosen by the host from the chunk counts alone so that at most
// kFinalizeMaxSlices slices exist).  One warp reduces one slice: lane l adds records
// l, l+32, ... of the slice in that order, four loads in flight, then a fixed shuffle tree;
// slices go round-robin to the warps of the cluster, and each partial is stored into CTA 0's
// shared memory (distributed shared memory for the other CTAs).  After the cluster barrier
// (a hardware barrier between co-scheduled CTAs, not a spin on memory) CTA 0 adds, one warp
// per shard, the shard's slice partials in lane-strided order and a tree, and its thread 0
// adds the shard records in shard order, takes the decision (Algorithm 1: statistic T_k and
// the If/Else) and writes the header.  The shape of every sum depends only on the chunk
// counts, never on the number of CTAs or on which warp took which slice.
constexpr int kFinalizeThreads = 1024;
constexpr int kFinalizeWarps = kFinalizeThreads / 32;
constexpr int kFinalizeMaxCtas = 8;
constexpr int kFinalizeSlice = 128;       // records: 32 lanes x 4 loads in flight
constexpr int kFinalizeMaxSlices = 1024;  // 24 KB of partials in CTA 0
constexpr int kFinalizeSlicesPerCta = 16;  // another CTA (another SM's L2 port) per 16 slices

// More than kInlineWorkers workers (up to ABS_MAX_WORKERS): the run-time loop of the kernel
// above over a pointer table that arrives as a second kernel parameter.
template <typename GT, bool ADAM, int STAT>
__global__ void __launch_bounds__(kThreads, 2)
    normtest_split_wide_kernel(const __grid_constant__ StreamParams prm,
                               const __grid_constant__ WideTable table) {
  __shared__ double red[kWarps * 3];
  const int K = prm.K;
  bool waited = false;
  GradWeights gw{prm.adam.omb1, prm.adam.omb2};
  for (int chunk = blockIdx.x; chunk < prm.n_chunks; chunk += gridDim.x) {
    const ChunkGeometry cg =
        chunk_geometry<GT, kInlineWorkers, false, ADAM>(prm, table.ptrs, K, chunk);
    if (!waited) {
      grid_dependency_wait();
      waited = true;
      if (ADAM) gw = grad_weights(prm.adam, prm.clip_n2, prm.clip_max_norm);
    }
    double acc_n2 = 0.0, acc_S = 0.0, acc_Q = 0.0;
    CwMax cw;
    cw.init(static_cast<int>(threadIdx.x) * GT::kVec);
    chunk_rows_split<GT, kInlineWorkers, false, ADAM, STAT>(prm, table.ptrs, K, cg, acc_n2, acc_S,
                                                            acc_Q, cw, gw);
    write_chunk_record<STAT>(prm, chunk, cg.lo, acc_n2, acc_S, acc_Q, cw, red);
  }
}

// records c0 + first, c0 + first + stride, ... (< c1), added in that order.  Each pass issues
// four unconditional loads (an index past the end re-reads the pass's first record and its
// values are replaced by +0.0, which leaves the sums unchanged) before the first add.
// CW: the third and fourth slot of a record are {index, ratio} of the chunk's largest
// per-coordinate ratio; (c, m) then carry the running {index, ratio} maximum instead of a sum.
template <bool CW>
__device__ __forceinline__ void strided_records(const double* chunk_in, int c0, int c1, int first,
                                                int stride, double& a, double& b, double& c,
                                                double& m) {
  constexpr int kInFlight = 4;
  for (int ch = c0 + first; ch < c1; ch += kInFlight * stride) {
    double2 t[kInFlight], u2[kInFlight];
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) {
      const int r = ch + u * stride;
      const double* rec = chunk_in + static_cast<int64_t>(r < c1 ? r : ch) * 4;
      t[u] = __ldcg(reinterpret_cast<const double2*>(rec));
      u2[u] = __ldcg(reinterpret_cast<const double2*>(rec + 2));
    }
#pragma unroll
    for (int u = 0; u < kInFlight; ++u) {
      const bool live = ch + u * stride < c1;
      a += live ? t[u].x : 0.0;
      b += live ? t[u].y : 0.0;
      if (CW) {
        if (live && (u2[u].y > m || (u2[u].y == m && u2[u].x < c))) {
          m = u2[u].y;
          c = u2[u].x;
        }
      } else {
        c += live ? u2[u].x : 0.0;
      }
    }
  }
}

template <bool CW>
__device__ __forceinline__ void warp_tree3(double& a, double& b, double& c, double& m) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    a += __shfl_down_sync(0xffffffffu, a, off);
    b += __shfl_down_sync(0xffffffffu, b, off);
    const double c2 = __shfl_down_sync(0xffffffffu, c, off);
    if (CW) {
      const double m2 = __shfl_down_sync(0xffffffffu, m, off);
      if (m2 > m || (m2 == m && c2 < c)) {
        m = m2;
        c = c2;
      }
    } else {
      c += c2;
    }
  }
}

// The decision of the coordinate-wise test from the largest per-coordinate ratio
// rmax = max_i sum_k (g_k[i]-gbar_i)^2 / gbar_i^2:  T = (rmax/norm) / eta^2.
__device__ __forceinline__ int64_t decide_coordwise_device(double S, double n2, double rmax,
                                                           double norm, double eta, int64_t b_cur,
                                                           double* T_out, int* flags_out) {
  int flags = 0;
  double T = (rmax / norm) / (eta * eta);
  int64_t b_next = b_cur;
  if (!isfinite(S) || !isfinite(n2)) {
    flags |= ABS_FLAG_NONFINITE;
    T = __longlong_as_double(0x7ff8000000000000ll);
  } else {
    if (n2 == 0.0 || isinf(T)) flags |= ABS_FLAG_DEGENERATE;
    if (T > static_cast<double>(b_cur)) {
      flags |= ABS_FLAG_VIOLATED;
      b_next = (T >= 4611686018427387904.0) ? INT64_MAX : static_cast<int64_t>(ceil(T));
    }
  }
  *T_out = T;
  *flags_out = flags;
  return b_next;
}

// CW: the coordinate-wise test (chunk records carry {n2, S, index, ratio}); the shard records
// written are {n2_s, S_s, index of the shard's largest T_i, that T_i}, the header's Q slot
// reads NaN, its T slot the largest T_i and its ABS_STAT_ARGMAX slot where it occurs.
template <bool CW>
__global__ void __launch_bounds__(kFinalizeThreads)
    finalize_kernel(const __grid_constant__ FinalizeParams fp) {
  namespace cg = cooperative_groups;
  constexpr int PS = CW ? 4 : 3;                    // doubles per partial
  __shared__ double part[kFinalizeMaxSlices * PS];  // used in CTA 0 only
  __shared__ double shard_tot[ABS_MAX_SHARDS * PS];
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = static_cast<int>(cluster.block_rank());
  const int n_warps = static_cast<int>(cluster.num_blocks()) * kFinalizeWarps;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  double* part0 = cluster.map_shared_rank(part, 0);
  const int n_slices = fp.slice_prefix[fp.n_shards];
  // Distributed shared memory of another CTA may only be touched once that CTA is known to
  // have started: every CTA of the cluster arrives here before the first remote store below.
  // The barrier touches no global memory, so it sits before the dependency wait and overlaps
  // the tail of the preceding kernel.
  cluster.sync();
  // This kernel occupies at most eight SMs: the next kernel of the stream (with the library's
  // calls back to back, the next call's streaming kernel) may be scheduled now and run up to its
  // own dependency wait -- which still holds it until this grid has completed -- so its launch and
  // prologue are off the critical path (0.5-0.6 us per call: d = 1M 10.4 -> 9.8 us).
  grid_launch_dependents();
  grid_dependency_wait();
  for (int i = rank * kFinalizeWarps + warp; i < n_slices; i += n_warps) {
    // the shard of slice i: the last s with slice_prefix[s] <= i
    int lo = 0, hi = fp.n_shards;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (fp.slice_prefix[mid] <= i) lo = mid; else hi = mid;
    }
    const int c0 = fp.chunk_prefix[lo] + (i - fp.slice_prefix[lo]) * fp.slice;
    const int c1 = min(c0 + fp.slice, fp.chunk_prefix[lo + 1]);
    double a = 0.0, b = 0.0, c = 0.0, m = -1.0;
    strided_records<CW>(fp.chunk_in, c0, c1, lane, 32, a, b, c, m);
    warp_tree3<CW>(a, b, c, m);
    if (lane == 0) {
      part0[PS * i + 0] = a;
      part0[PS * i + 1] = b;
      part0[PS * i + 2] = c;
      if (CW) part0[PS * i + 3] = m;
    }
  }
  // arrive.release / wait.acquire at cluster scope: every partial is visible to CTA 0
  cluster.sync();
  if (rank != 0) return;
  for (int s = warp; s < fp.n_shards; s += kFinalizeWarps) {
    double a = 0.0, b = 0.0, c = 0.0, m = -1.0;
    for (int i = fp.slice_prefix[s] + lane; i < fp.slice_prefix[s + 1]; i += 32) {
      a += part[PS * i + 0];
      b += part[PS * i + 1];
      if (CW) {
        const double m2 = part[PS * i + 3], c2 = part[PS * i + 2];
        if (m2 > m || (m2 == m && c2 < c)) {
          m = m2;
          c = c2;
        }
      } else {
        c += part[PS * i + 2];
      }
    }
    warp_tree3<CW>(a, b, c, m);
    if (lane == 0) {
      double* rec = fp.stats + ABS_STATS_HEADER + s * ABS_SHARD_STRIDE;
      rec[0] = a;
      rec[1] = b;
      if (CW) {
        // an empty shard has no coordinate: ratio 0 at its (empty) start
        if (m < 0.0) {
          m = 0.0;
          c = static_cast<double>(fp.shard_first[s]);
        }
        rec[2] = c;
        rec[3] = (m / fp.norm) / (fp.eta * fp.eta);
      } else {
        rec[2] = c;
        rec[3] = 0.0;
      }
      shard_tot[PS * s + 0] = a;
      shard_tot[PS * s + 1] = b;
      shard_tot[PS * s + 2] = c;
      if (CW) shard_tot[PS * s + 3] = m;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double tot_n2 = 0.0, tot_S = 0.0, tot_Q = 0.0, rmax = 0.0, arg = 0.0;
    bool any = false;
    for (int s = 0; s < fp.n_shards; ++s) {
      tot_n2 += shard_tot[PS * s + 0];
      tot_S += shard_tot[PS * s + 1];
      if (CW) {
        // shards in index order: a later shard wins only with a strictly larger ratio, so a
        // tie keeps the lower coordinate; empty shards do not take part
        const bool nonempty = fp.chunk_prefix[s + 1] > fp.chunk_prefix[s];
        if (nonempty && (!any || shard_tot[PS * s + 3] > rmax)) {
          rmax = shard_tot[PS * s + 3];
          arg = shard_tot[PS * s + 2];
          any = true;
        }
      } else {
        tot_Q += shard_tot[PS * s + 2];
      }
    }
    double T;
    int flags;
    int64_t b_next;
    if (CW) {
      b_next = decide_coordwise_device(tot_S, tot_n2, rmax, fp.norm, fp.eta, fp.b_cur, &T, &flags);
      tot_Q = __longlong_as_double(0x7ff8000000000000ll);
    } else {
      b_next = decide_device(tot_S, tot_n2, fp.norm, fp.eta, fp.b_cur, &T, &flags);
    }
    fp.stats[ABS_STAT_N2] = tot_n2;
    fp.stats[ABS_STAT_S] = tot_S;
    fp.stats[ABS_STAT_Q] = tot_Q;
    fp.stats[ABS_STAT_T] = T;
    fp.stats[ABS_STAT_FLAGS] = static_cast<double>(flags);
    fp.stats[ABS_STAT_NORM] = fp.norm;
    fp.stats[ABS_STAT_NCHUNKS] = static_cast<double>(fp.n_chunks);
    fp.stats[ABS_STAT_ARGMAX] = CW ? arg : 0.0;
    *fp.b_next = b_next;
  }
}

}  // namespace absnt
