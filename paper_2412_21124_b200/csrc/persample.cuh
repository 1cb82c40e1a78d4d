// Per-sample form of the norm test (Eq. 3 with the Var definition before it): column
// mean and column sum of squared deviations of a row-major [b, ld] matrix whose rows
// are per-sample gradients (fp32 or bf16), reading the matrix once.
//
// Pass 1 (2-D grid: column block x row block): a thread owns 4 adjacent columns and walks its
// row block in groups of kGroup rows.  Each value is consumed once: per group and column the
// thread accumulates sum(x) in fp64 (exact for any realistic spread of fp32 or bf16 values)
// and, about a centre c close to the column mean (the first row for the first
// group, the running mean afterwards), sum((x-c)^2) in fp32; then
//     M2_g = sum((x-c)^2) - n_g (sum_g/n_g - c)^2                      (shift identity)
// and the group is merged into the running {sum, M2} of the column in sum form,
//     M2 += M2_g + (n sum_g - n_g sum)^2 / (n n_g (n + n_g));   sum += sum_g
// (law of total variance).  Sums, not means, are carried: the column mean is then one division
// of an fp64 sum at the very end, so rows that cancel exactly give a mean of exactly zero.
// How the rows arrive: every thread keeps kRing rows of its own 16 (8) bytes in flight with
// cp.async into a ring in shared memory that only it reads -- no barrier anywhere -- which
// keeps 3 CTAs x 128 threads x 16 rows x 16 B = 98 KB in flight per SM at 127 registers per
// thread (rows held in registers managed 49 KB at 161 registers).  Matrices whose rows are
// not 16-byte (8-byte) aligned take the same arithmetic with plain element loads.
// It writes {sum, M2} per (row block, column).
// Pass 2 (one thread per column, 128 columns per CTA) merges the row blocks: the column sum
// (row blocks added in index order) gives the mean, then
//     M2 = sum_rb [ M2_rb + n_rb (sum_rb/n_rb - mean)^2 ]                  (same order)
// -- no serial chain, all records of a column in flight at once.  It writes gbar and reduces
// {gbar^2, M2} over its columns in a fixed order into the CTA's record.  The decision needs
// the sum over all CTAs: each CTA, having published its record, draws a ticket (one atomic
// add; no CTA ever waits for another), and the CTA that draws the last ticket adds the records
// in index order, takes the decision (Eq. 3 and the display after it) and writes the header.
// Which CTA does that depends on timing, what it computes does not.  The ticket counter is put
// back to zero by the CTA that drew the last ticket, so a stats buffer that starts zero-filled
// stays usable call after call.
// Why two launches and not one or three: folding the merge into pass 1 with one more level of
// tickets makes every streaming CTA sit on its SM through two or three loaded memory round
// trips before it can leave (measured: 41.9 us of streaming became 59 us); a third launch for
// the final sum costs another drain and launch (2.7 us) where the ticket costs one round trip.
// The diagnostic Q is not computed by this call (its slots read NaN).
// Also here: the stand-alone AdamW kernel.
#pragma once
#include <type_traits>

#include "normtest_stream.cuh"

namespace absnt {

constexpr int kGroup = 16;        // rows per group (one shift centre, one merge)
constexpr int kBatch = 8;         // rows per cp.async commit group
#ifndef ABS_PS_RING_BATCHES
#define ABS_PS_RING_BATCHES 2
#endif
#ifndef ABS_PS_CTAS_PER_SM
#define ABS_PS_CTAS_PER_SM 3
#endif
// Measured, whole call, fp32 (b x d = 4096 x 16384, 268 MB, one wave / 4096 x 65536, 1.07 GB):
// 3 CTAs per SM x 16 rows in flight per thread 46.9 / 163.2 us; 2 x 32 rows 47.5 / 171.5;
// 2 x 24 rows 46.8 / 172.9; 3 x 24 rows 48.7 / 172.3; 4 x 16 rows 50.6 / 164.5.  More rows in
// flight than about 16 per thread at three or four CTAs per SM do not pay: 20 MB in flight on
// the device is past what the memory system rewards.
constexpr int kRingBatches = ABS_PS_RING_BATCHES;  // batches in flight per thread
constexpr int kRing = kBatch * kRingBatches;
constexpr int kPsThreads = 128;                    // threads per CTA of the per-sample kernel
constexpr int kPsCtasPerSM = ABS_PS_CTAS_PER_SM;

struct PersampleParams {
  const void* G;
  int64_t b, d, ld;
  int rows_per_block;
  int n_row_blocks;
  double* ws_sum;  // [n_row_blocks][d]
  double* ws_m2;
  float* gbar;
  double* cb_rec;         // kPsRecDoubles per CTA of pass 2 (kPsThreads columns): {n2, S, largest
                          // per-column ratio, its column} -- the last two in the coordinate-wise form
  unsigned int* tickets;  // one counter, zero at entry and again on return
  double* stats;          // header + one shard record
  int64_t* b_next;
  double eta;
};

// element types of the matrix: 4 columns of a thread are one PsVec
struct PsF32 {
  using scalar = float;
  using vec = uint4;
  using gsum_t = double;  // group sums of fp32 values need fp64 to stay exact
  static __device__ __forceinline__ void unpack(const vec& r, float (&x)[4]) {
    x[0] = __uint_as_float(r.x);
    x[1] = __uint_as_float(r.y);
    x[2] = __uint_as_float(r.z);
    x[3] = __uint_as_float(r.w);
  }
  static __device__ __forceinline__ float load1(const void* p) {
    return __ldg(reinterpret_cast<const float*>(p));
  }
};
struct PsBF16 {
  using scalar = uint16_t;
  using vec = uint2;
  using gsum_t = double;  // as for fp32: exact sums whatever the spread of the 16 values
  static __device__ __forceinline__ void unpack(const vec& r, float (&x)[4]) {
    x[0] = bf16_lo(r.x);
    x[1] = bf16_hi(r.x);
    x[2] = bf16_lo(r.y);
    x[3] = bf16_hi(r.y);
  }
  static __device__ __forceinline__ float load1(const void* p) {
    return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const uint16_t*>(p)))
                           << 16);
  }
};

// global -> this thread's slot of the ring; `src_bytes` < sizeof(vec) zero-fills the rest
template <typename ET>
__device__ __forceinline__ void ps_async_copy(void* smem_dst, const void* src, int src_bytes) {
  const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
  if constexpr (sizeof(typename ET::vec) == 16)
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src),
                 "r"(src_bytes)
                 : "memory");
  else
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src),
                 "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void ps_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void ps_wait_pending() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// running {sum, M2, count} of one column and the merge of a group / row block into it
struct PsColumn {
  double sum, m2;
};
__device__ __forceinline__ void ps_merge(PsColumn& a, int64_t n, double sum_g, double m2_g,
                                         int64_t n_g, double coef /* 1/(n n_g (n+n_g)) */) {
  if (n == 0) {
    a.sum = sum_g;
    a.m2 = m2_g;
  } else {
    const double t = static_cast<double>(n) * sum_g - static_cast<double>(n_g) * a.sum;
    a.m2 += m2_g + (t * t) * coef;
    a.sum += sum_g;
  }
}
__device__ __forceinline__ double ps_coef(int64_t n, int64_t n_g) {
  const double dn = static_cast<double>(n), dg = static_cast<double>(n_g);
  return n == 0 ? 0.0 : 1.0 / (dn * dg * (dn + dg));
}

template <typename ET, bool RING>
__global__ void __launch_bounds__(kPsThreads, kPsCtasPerSM)
    persample_partial_kernel(const __grid_constant__ PersampleParams prm) {
  using Vec = typename ET::vec;
  constexpr int ES = static_cast<int>(sizeof(typename ET::scalar));
  extern __shared__ __align__(16) unsigned char ps_ring_raw[];
  Vec* ring = reinterpret_cast<Vec*>(ps_ring_raw);  // [kRing][kPsThreads], RING only
  const int tid = threadIdx.x;
  const int64_t c0 = (static_cast<int64_t>(blockIdx.x) * kPsThreads + tid) * 4;
  grid_dependency_wait();
  const bool active = c0 < prm.d;  // the last column block may have threads without columns
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * prm.rows_per_block;
  const int64_t r1 = (r0 + prm.rows_per_block < prm.b) ? r0 + prm.rows_per_block : prm.b;
  const int nrows = static_cast<int>(r1 - r0);
  const int live_cols = !active ? 0 : ((prm.d - c0 < 4) ? static_cast<int>(prm.d - c0) : 4);
  const unsigned char* base = static_cast<const unsigned char*>(prm.G) +
                              (r0 * prm.ld + c0) * ES;
  const int64_t stride = prm.ld * ES;

  // row i of the block (0-based) into x: from the ring, or with plain element loads
  auto issue_batch = [&](int first_row) {  // rows first_row .. first_row + kBatch - 1
    if constexpr (RING) {
#pragma unroll
      for (int j = 0; j < kBatch; ++j) {
        const int i = first_row + j;
        if (i < nrows)
          ps_async_copy<ET>(&ring[(i % kRing) * kPsThreads + tid], base + i * stride,
                            live_cols * ES);
      }
      ps_commit();
    }
  };
  auto fetch_row = [&](int i, float (&x)[4]) {
    if constexpr (RING) {
      ET::unpack(ring[(i % kRing) * kPsThreads + tid], x);
    } else {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        x[q] = (q < live_cols) ? ET::load1(base + i * stride + q * ES) : 0.f;
    }
  };

  PsColumn col[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) col[q].sum = col[q].m2 = 0.0;
  int64_t n = 0;

  // one group of ng rows starting at block row g0; FULL: ng == kGroup (no row predicates)
  auto group = [&](int g0, int ng, auto full_tag) {
    constexpr bool FULL = decltype(full_tag)::value;
    typename ET::gsum_t s0[4], s1[4];
    float c[4], s2[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      s0[q] = s1[q] = 0;
      s2[q] = 0.f;
    }
    const double inv_n = (n == 0) ? 0.0 : 1.0 / static_cast<double>(n);
#pragma unroll
    for (int half = 0; half < kGroup / kBatch; ++half) {
      const int h0 = g0 + half * kBatch;
      if (RING) ps_wait_pending<kRingBatches - 1>();  // this batch has landed
      float x[kBatch][4];
#pragma unroll
      for (int j = 0; j < kBatch; ++j)
        if (FULL || h0 + j < nrows) fetch_row(h0 + j, x[j]);
      // the slots just read are free: the batch kRing rows ahead goes into them
      issue_batch(h0 + kRing);
      if (half == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
          c[q] = (n == 0) ? x[0][q] : static_cast<float>(col[q].sum * inv_n);
      }
#pragma unroll
      for (int j = 0; j < kBatch; ++j) {
        if (FULL || h0 + j < nrows) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float v = x[j][q];
            if (j & 1) s1[q] += static_cast<typename ET::gsum_t>(v);
            else s0[q] += static_cast<typename ET::gsum_t>(v);
          }
          // deviations and their squares two columns at a time (packed fp32: each lane rounds
          // like the scalar instruction; the bf16 kernel is bound by instruction issue and gains
          // 26% from it, 51.2 -> 40.7 us at b = 4096, d = 16384; the fp32 kernel is unchanged)
#pragma unroll
          for (int qp = 0; qp < 2; ++qp) {
            const float2 dv = __fadd2_rn(make_float2(x[j][2 * qp], x[j][2 * qp + 1]),
                                         make_float2(-c[2 * qp], -c[2 * qp + 1]));
            const float2 acc = __ffma2_rn(dv, dv, make_float2(s2[2 * qp], s2[2 * qp + 1]));
            s2[2 * qp] = acc.x;
            s2[2 * qp + 1] = acc.y;
          }
        }
      }
    }
    const double dg = static_cast<double>(ng);
    const double coef = ps_coef(n, ng);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const double sum_g = static_cast<double>(s0[q]) + static_cast<double>(s1[q]);
      // a power-of-two count divides exactly by multiplication
      const double mu = FULL ? sum_g * (1.0 / kGroup) : sum_g / dg;
      const double dc = mu - static_cast<double>(c[q]);
      const double m2g = clamp_nonneg(static_cast<double>(s2[q]) - dg * dc * dc);
      ps_merge(col[q], n, sum_g, m2g, ng, coef);
    }
    n += ng;
  };
  if (active) {
#pragma unroll
    for (int bt = 0; bt < kRingBatches; ++bt) issue_batch(bt * kBatch);
    const int n_full = nrows / kGroup;
    for (int gi = 0; gi < n_full; ++gi) group(gi * kGroup, kGroup, std::true_type{});
    if (n_full * kGroup < nrows)  // the last, ragged group of the row block
      group(n_full * kGroup, nrows - n_full * kGroup, std::false_type{});
    if (RING) ps_wait_pending<0>();
  }
  // this row block's records; the CTA leaves at once (nothing here waits on memory)
  const int64_t o = static_cast<int64_t>(blockIdx.y) * prm.d + c0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    if (q < live_cols) {
      __stcg(prm.ws_sum + o + q, col[q].sum);
      __stcg(prm.ws_m2 + o + q, col[q].m2);
    }
  }
}

// Pass 2 and the decision (see the top of the file).
constexpr int kPsTicketDoubles = 2;    // room for the ticket counter in stats_out (keeps 16-byte alignment)
constexpr int kPsMergeInFlight = 16;  // row blocks of a column in flight at once
constexpr int kPsRecDoubles = 4;      // doubles per record of a merge CTA

// The running maximum of {ratio, column} with ties to the lower column; a NaN ratio never wins.
__device__ __forceinline__ void ps_take_max(double& r, double& idx, double r2, double idx2) {
  if (r2 > r || (r2 == r && idx2 < idx)) {
    r = r2;
    idx = idx2;
  }
}
__device__ __forceinline__ void ps_block_max(double& r, double& idx, double* sm /* 2 per warp */) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const double r2 = __shfl_down_sync(0xffffffffu, r, off);
    const double i2 = __shfl_down_sync(0xffffffffu, idx, off);
    ps_take_max(r, idx, r2, i2);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    sm[2 * warp] = r;
    sm[2 * warp + 1] = idx;
  }
  __syncthreads();
  if (threadIdx.x == 0)
    for (int w = 1; w < kPsThreads / 32; ++w) ps_take_max(r, idx, sm[2 * w], sm[2 * w + 1]);
  __syncthreads();
}

// CW: the coordinate-wise test in its per-sample form (Sec. 4, Proposition 1, with the sample
// variance of the Var definition before Eq. 3): per column i the ratio M2_i / gbar_i^2 (zero when
// M2_i = 0, +inf when only gbar_i = 0), the decision from the largest one,
// T = (max_i ratio_i / (b-1)) / eta^2, and the column where it occurs.
template <bool CW>
__global__ void __launch_bounds__(kPsThreads)
    persample_merge_kernel(const __grid_constant__ PersampleParams prm) {
  __shared__ double red[(kPsThreads / 32) * 3];
  __shared__ double red_max[(kPsThreads / 32) * 2];
  __shared__ int s_last;
  const int tid = threadIdx.x;
  const int64_t c = static_cast<int64_t>(blockIdx.x) * kPsThreads + tid;
  const int nrb = prm.n_row_blocks;
  const int64_t n_last = prm.b - static_cast<int64_t>(nrb - 1) * prm.rows_per_block;
  const double n_full = static_cast<double>(prm.rows_per_block);
  const double inv_full = 1.0 / n_full, inv_last = 1.0 / static_cast<double>(n_last);
  // a small grid: the next kernel of the stream may be scheduled and run up to its own
  // dependency wait (b = 4096, d = 16384: 46.8 -> 46.4 us per call; b = 256: 10.9 -> 11.1)
  grid_launch_dependents();
  grid_dependency_wait();
  double a = 0.0, sdev = 0.0, unused = 0.0;
  double rmax = -1.0, rarg = static_cast<double>(c);  // -1: no column (or only NaN ratios) yet
  if (c < prm.d) {
    double su[kPsMergeInFlight], mm[kPsMergeInFlight];
    double tot = 0.0;
    if (nrb <= kPsMergeInFlight) {
      // the usual case: every record of the column is loaded once and kept
#pragma unroll
      for (int u = 0; u < kPsMergeInFlight; ++u) {
        const int64_t o = static_cast<int64_t>(u < nrb ? u : 0) * prm.d + c;
        su[u] = (u < nrb) ? __ldcg(prm.ws_sum + o) : 0.0;
        mm[u] = (u < nrb) ? __ldcg(prm.ws_m2 + o) : 0.0;
      }
#pragma unroll
      for (int u = 0; u < kPsMergeInFlight; ++u) tot += su[u];
    } else {
      for (int rb0 = 0; rb0 < nrb; rb0 += kPsMergeInFlight) {
#pragma unroll
        for (int u = 0; u < kPsMergeInFlight; ++u) {
          const int64_t o = static_cast<int64_t>(rb0 + u < nrb ? rb0 + u : 0) * prm.d + c;
          su[u] = (rb0 + u < nrb) ? __ldcg(prm.ws_sum + o) : 0.0;
        }
#pragma unroll
        for (int u = 0; u < kPsMergeInFlight; ++u) tot += su[u];
      }
    }
    // the column mean: one division of the fp64 column sum (identical rows give their common
    // value exactly, rows that cancel give exactly zero)
    const double mean = tot / static_cast<double>(prm.b);
    double m2 = 0.0;
    for (int rb0 = 0; rb0 < nrb; rb0 += kPsMergeInFlight) {
      if (nrb > kPsMergeInFlight) {
#pragma unroll
        for (int u = 0; u < kPsMergeInFlight; ++u) {
          const int64_t o = static_cast<int64_t>(rb0 + u < nrb ? rb0 + u : 0) * prm.d + c;
          su[u] = (rb0 + u < nrb) ? __ldcg(prm.ws_sum + o) : 0.0;
          mm[u] = (rb0 + u < nrb) ? __ldcg(prm.ws_m2 + o) : 0.0;
        }
      }
#pragma unroll
      for (int u = 0; u < kPsMergeInFlight; ++u) {
        const int rb = rb0 + u;
        if (rb < nrb) {
          const bool last = rb == nrb - 1;
          const double nb = last ? static_cast<double>(n_last) : n_full;
          // (sum_rb - n_rb mean) / n_rb: the numerator is exact for identical rows, so they
          // contribute exactly zero
          const double dmu = fma(-nb, mean, su[u]) * (last ? inv_last : inv_full);
          m2 += mm[u] + nb * (dmu * dmu);
        }
      }
    }
    const float gb = static_cast<float>(mean);
    prm.gbar[c] = gb;
    a = static_cast<double>(gb) * static_cast<double>(gb);
    sdev = m2;
    if (CW) {
      const double ratio = (m2 == 0.0) ? 0.0 : m2 / (mean * mean);
      if (ratio > rmax) rmax = ratio;  // a NaN ratio leaves -1
    }
  }
  block_reduce3<kPsThreads / 32>(a, sdev, unused, red);
  if (CW) ps_block_max(rmax, rarg, red_max);
  // One fence per CTA: thread 0 wrote the record itself; its fence publishes it before the
  // ticket is drawn, and on the winning side it fences again before the barrier releases the
  // CTA to read the other records.
  if (tid == 0) {
    double* rec = prm.cb_rec + kPsRecDoubles * static_cast<int64_t>(blockIdx.x);
    __stcg(rec, a);
    __stcg(rec + 1, sdev);
    if (CW) {
      __stcg(rec + 2, rmax);
      __stcg(rec + 3, rarg);
    }
    __threadfence();
    s_last = atomicAdd(prm.tickets, 1u) == gridDim.x - 1u;
    if (s_last) __threadfence();
  }
  __syncthreads();
  if (!s_last) return;

  // records in index order: thread t takes t, t + 128, ...; then the fixed tree
  double n2 = 0.0, S = 0.0;
  rmax = -1.0;
  rarg = 0.0;
  for (int64_t cb = tid; cb < static_cast<int64_t>(gridDim.x); cb += kPsThreads) {
    const double* rec = prm.cb_rec + kPsRecDoubles * cb;
    n2 += __ldcg(rec);
    S += __ldcg(rec + 1);
    if (CW) ps_take_max(rmax, rarg, __ldcg(rec + 2), __ldcg(rec + 3));
  }
  block_reduce3<kPsThreads / 32>(n2, S, unused, red);
  if (CW) ps_block_max(rmax, rarg, red_max);
  if (tid == 0) {
    const double norm = static_cast<double>(prm.b - 1);
    double T;
    int flags;
    if (CW && rmax < 0.0) {  // every ratio was NaN: the sums are non-finite and say so
      rmax = 0.0;
      rarg = 0.0;
    }
    const int64_t b_next =
        CW ? decide_coordwise_device(S, n2, rmax, norm, prm.eta, prm.b, &T, &flags)
           : decide_device(S, n2, norm, prm.eta, prm.b, &T, &flags);
    const double nan = __longlong_as_double(0x7ff8000000000000ll);
    prm.stats[ABS_STAT_N2] = n2;
    prm.stats[ABS_STAT_S] = S;
    prm.stats[ABS_STAT_Q] = nan;  // not computed
    prm.stats[ABS_STAT_T] = T;
    prm.stats[ABS_STAT_FLAGS] = static_cast<double>(flags);
    prm.stats[ABS_STAT_NORM] = norm;
    prm.stats[ABS_STAT_NCHUNKS] = static_cast<double>(gridDim.x);
    prm.stats[ABS_STAT_ARGMAX] = CW ? rarg : 0.0;
    double* rec = prm.stats + ABS_STATS_HEADER;  // the one shard record
    rec[0] = n2;
    rec[1] = S;
    rec[2] = CW ? rarg : nan;
    rec[3] = CW ? T : 0.0;
    *prm.b_next = b_next;
    *prm.tickets = 0u;  // ready for the next call
  }
}

// Stand-alone AdamW (Algorithm 1, AdamW lines), in place, for vectors below 2^25 coordinates
// (larger ones run as the one-worker fused kernel).  With `n2_dev` non-null the
// gradient is first clipped by global norm: g <- g * min(1, max_norm / (sqrt(n2) + 1e-6)),
// n2 = ||gbar||^2 read from the stats header a preceding norm test wrote on the device
// (no host round trip).  Clipping is what the paper's experiments add to Algorithm 1.
template <bool VEC>
__global__ void __launch_bounds__(kThreads)
    adamw_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m,
                 float* __restrict__ v, int64_t d, const AdamScalars a,
                 const double* __restrict__ n2_dev, double max_norm, uint16_t* __restrict__ p16) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  grid_dependency_wait();
  // the clipping scale is folded into the weights of the new gradient (see GradWeights)
  const GradWeights gw = grad_weights(a, n2_dev, max_norm);
  if (VEC) {
    const int64_t nvec = d >> 2;
    int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x;
    // two vectors per array in flight per thread
    for (; i + stride < nvec; i += 2 * stride) {
      const int64_t j = i + stride;
      const float4 g0 = __ldcs(reinterpret_cast<const float4*>(g) + i);
      const float4 g1 = __ldcs(reinterpret_cast<const float4*>(g) + j);
      float4 p0 = ld_state_16(p + 4 * i), m0 = ld_state_16(m + 4 * i), v0 = ld_state_16(v + 4 * i);
      float4 p1 = ld_state_16(p + 4 * j), m1 = ld_state_16(m + 4 * j), v1 = ld_state_16(v + 4 * j);
      adamw_elem(a, gw.omb1, gw.omb2, g0.x, p0.x, m0.x, v0.x);
      adamw_elem(a, gw.omb1, gw.omb2, g0.y, p0.y, m0.y, v0.y);
      adamw_elem(a, gw.omb1, gw.omb2, g0.z, p0.z, m0.z, v0.z);
      adamw_elem(a, gw.omb1, gw.omb2, g0.w, p0.w, m0.w, v0.w);
      st_stream_16(p + 4 * i, p0);
      st_stream_16(m + 4 * i, m0);
      st_stream_16(v + 4 * i, v0);
      if (p16) st_bf16x4(p16 + 4 * i, p0);
      adamw_elem(a, gw.omb1, gw.omb2, g1.x, p1.x, m1.x, v1.x);
      adamw_elem(a, gw.omb1, gw.omb2, g1.y, p1.y, m1.y, v1.y);
      adamw_elem(a, gw.omb1, gw.omb2, g1.z, p1.z, m1.z, v1.z);
      adamw_elem(a, gw.omb1, gw.omb2, g1.w, p1.w, m1.w, v1.w);
      st_stream_16(p + 4 * j, p1);
      st_stream_16(m + 4 * j, m1);
      st_stream_16(v + 4 * j, v1);
      if (p16) st_bf16x4(p16 + 4 * j, p1);
    }
    if (i < nvec) {
      const float4 gg = __ldcs(reinterpret_cast<const float4*>(g) + i);
      float4 pp = ld_state_16(p + 4 * i), mm = ld_state_16(m + 4 * i), vv = ld_state_16(v + 4 * i);
      adamw_elem(a, gw.omb1, gw.omb2, gg.x, pp.x, mm.x, vv.x);
      adamw_elem(a, gw.omb1, gw.omb2, gg.y, pp.y, mm.y, vv.y);
      adamw_elem(a, gw.omb1, gw.omb2, gg.z, pp.z, mm.z, vv.z);
      adamw_elem(a, gw.omb1, gw.omb2, gg.w, pp.w, mm.w, vv.w);
      st_stream_16(p + 4 * i, pp);
      st_stream_16(m + 4 * i, mm);
      st_stream_16(v + 4 * i, vv);
      if (p16) st_bf16x4(p16 + 4 * i, pp);
    }
    // tail (d % 4 elements) by the first threads of block 0
    const int64_t t = (nvec << 2) + threadIdx.x;
    if (blockIdx.x == 0 && t < d) {
      float pp = p[t], mm = m[t], vv = v[t];
      adamw_elem(a, gw.omb1, gw.omb2, g[t], pp, mm, vv);
      p[t] = pp;
      m[t] = mm;
      v[t] = vv;
      if (p16) p16[t] = to_bf16(pp);
    }
  } else {
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < d;
         i += stride) {
      float pp = p[i], mm = m[i], vv = v[i];
      adamw_elem(a, gw.omb1, gw.omb2, g[i], pp, mm, vv);
      p[i] = pp;
      m[i] = mm;
      v[i] = vv;
      if (p16) p16[i] = to_bf16(pp);
    }
  }
}

}  // namespace absnt
