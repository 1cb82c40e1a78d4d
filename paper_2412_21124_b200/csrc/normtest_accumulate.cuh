// Carry-in form of the norm test: the worker (or micro-batch) gradients of one step arrive a
// few at a time -- as they do under gradient accumulation -- and are merged into a running
// state of O(d) memory instead of being kept side by side.
//
// State between the calls of a step: the running mean of the n gradients merged so far (d fp32
// values: the gradient-accumulation buffer itself, holding the mean instead of the sum) and, per
// shard, the running sum of squared deviations about that mean (in the shard records of the
// stats buffer).  Merging m new gradients g_1..g_m into (n, mean, M2), per coordinate, with the
// old mean as the centre c (for n = 0: c = g_1):
//     sd = sum_k (g_k - c)        q = sum_k (g_k - c)^2
//     mean' = c + sd / (n + m)    M2' = M2 + q - sd^2 / (n + m)
// which is the pooled-variance update (law of total variance) written about the old mean: the
// term taken off q is never larger than q (Cauchy-Schwarz) and small against it once n >> m,
// so nothing cancels.  After the last call mean' is gbar of Algorithm 1 ("Compute the batch
// gradient"), sum_i M2'_i the variance sum of Eq. 5, and n2 = sum_i mean'_i^2 is recomputed by
// every call (each call visits every coordinate).  Deviations and their squares are fp32 per
// coordinate, accumulated per group of workers and then over groups (as in the many-worker
// kernel), fp64 from the thread-row upwards.
//
// The chunk records have the layout of the other streaming kernels and go through the same
// finalize kernel; the carry enters as one more addend: the CTA of a shard's first chunk adds
// the shard's previous sum to its own partial.  Few workers per call leave little in flight,
// so up to one group of workers (16 bf16 / 8 fp32) a thread loads several thread-rows, or two
// rows of the whole group, before it consumes the first (the kernel's ROWS and KR).
#pragma once
#include "normtest_stream.cuh"

namespace absnt {

struct AccumCarry {
  double n_prev;            // gradients merged by the earlier calls of this step; 0 starts a step
  float inv_total;          // 1 / (n_prev + K)
  const float* mean_in;     // running mean of those n_prev gradients (unused when n_prev = 0)
  const double* shard_rec;  // shard records left by the previous call (slot 1: its sum S_s)
};
// The new mean goes to prm.gbar (which may be mean_in itself).  The closing call of a step can
// run AdamW on it in the same pass (ADAM: prm.p, m, v, p16 as in the fused kernels); prm.gbar
// may then be null -- the mean is consumed in registers and not written.

// Accumulators of one thread-row (four coordinates as two packed pairs).
template <typename GT>
struct AccumRow {
  static constexpr int P = 2;
  float2 c[P], neg_c[P];  // the centre
  float2 s2[P], g2[P];    // squared deviations: closed groups, the open group
  float2 sd[P], gd[P];    // deviations: the same
  // the centre: the running mean, or (first call of a step) the first gradient, set by the caller
  __device__ __forceinline__ void init(const float4& centre) {
#pragma unroll
    for (int pi = 0; pi < P; ++pi) s2[pi] = g2[pi] = sd[pi] = gd[pi] = make_float2(0.f, 0.f);
    c[0] = make_float2(centre.x, centre.y);
    c[1] = make_float2(centre.z, centre.w);
#pragma unroll
    for (int pi = 0; pi < P; ++pi) neg_c[pi] = make_float2(-c[pi].x, -c[pi].y);
  }
  __device__ __forceinline__ void init_from(const typename GT::raw_t& first_gradient) {
    const float2 a = GT::pair(first_gradient, 0), b = GT::pair(first_gradient, 1);
    init(make_float4(a.x, a.y, b.x, b.y));
  }
  __device__ __forceinline__ void add(const typename GT::raw_t& raw) {
#pragma unroll
    for (int pi = 0; pi < P; ++pi) {
      const float2 dv = __fadd2_rn(GT::pair(raw, pi), neg_c[pi]);
      gd[pi] = __fadd2_rn(gd[pi], dv);
      g2[pi] = __ffma2_rn(dv, dv, g2[pi]);
    }
  }
  __device__ __forceinline__ void close_group() {
#pragma unroll
    for (int pi = 0; pi < P; ++pi) {
      s2[pi] = __fadd2_rn(s2[pi], g2[pi]);
      sd[pi] = __fadd2_rn(sd[pi], gd[pi]);
      g2[pi] = gd[pi] = make_float2(0.f, 0.f);
    }
  }
  // the new means of the four coordinates; adds their squares and the M2 increments
  __device__ __forceinline__ float4 finish(float inv_total, float& row_n2, float& row_S) {
    float mean[4];
#pragma unroll
    for (int pi = 0; pi < P; ++pi) {
      const float2 it = make_float2(inv_total, inv_total);
      const float2 dm = __fmul2_rn(sd[pi], it);
      const float2 mu = __fadd2_rn(c[pi], dm);
      const float2 t = __ffma2_rn(make_float2(-sd[pi].x, -sd[pi].y), dm, s2[pi]);
      mean[2 * pi] = mu.x;
      mean[2 * pi + 1] = mu.y;
      row_n2 = fmaf(mu.x, mu.x, row_n2);
      row_n2 = fmaf(mu.y, mu.y, row_n2);
      row_S += clamp_nonneg(t.x);
      row_S += clamp_nonneg(t.y);
    }
    return make_float4(mean[0], mean[1], mean[2], mean[3]);
  }
};

// One thread-row with element-wise, bounds-checked accesses (ragged end of a shard, streams
// that are not 16-byte aligned): the operations of AccumRow in the same order.
template <typename GT, bool ADAM>
__device__ __noinline__ void accumulate_scalar_row(const StreamParams& prm, const AccumCarry& cy,
                                                   int K, int64_t base, int64_t hi, float* sums) {
  constexpr int H = split_group<GT, false>();
  const bool carry = cy.n_prev > 0.0;
  float row_n2 = 0.f, row_S = 0.f;
  for (int e = 0; e < GT::kVec; ++e) {
    const int64_t i = base + e;
    if (i >= hi) break;
    const float c = carry ? cy.mean_in[i] : GT::load1(prm.grads[0], i);
    float s2 = 0.f, g2 = 0.f, sd = 0.f, gd = 0.f;
    for (int k = 0; k < K; ++k) {
      const float dv = GT::load1(prm.grads[k], i) - c;
      gd += dv;
      g2 = fmaf(dv, dv, g2);
      if ((k + 1) % H == 0 || k + 1 == K) {
        s2 += g2;
        sd += gd;
        g2 = gd = 0.f;
      }
    }
    const float dm = sd * cy.inv_total;
    const float mu = c + dm;
    row_n2 = fmaf(mu, mu, row_n2);
    row_S += clamp_nonneg(fmaf(-sd, dm, s2));
    if (prm.gbar) prm.gbar[i] = mu;
    if (ADAM) {
      float w = prm.p[i], m = prm.m[i], v = prm.v[i];
      adamw_elem(prm.adam, prm.adam.omb1, prm.adam.omb2, mu, w, m, v);
      prm.p[i] = w;
      prm.m[i] = m;
      prm.v[i] = v;
      if (prm.p16) prm.p16[i] = to_bf16(w);
    }
  }
  sums[0] = row_n2;
  sums[1] = row_S;
}

// KR > 1: the call has at most KR workers, whose loads are issued as one predicated batch.
// ROWS > 1: calls with at most KR workers load ROWS thread-rows (ROWS * K gradient vectors and the
// ROWS mean vectors: 128 bytes of gradients per thread for ROWS * KR = 8 vectors of 16 bytes or
// 16 of 8 bytes) before the first is consumed; rows are consumed in order, so the sums have the
// shape of the ROWS = 1 kernel and both give the same bits.
template <typename GT, int ROWS, int KR, bool ADAM>
__global__ void __launch_bounds__(
    kThreads, (ADAM || ROWS * KR * static_cast<int>(sizeof(typename GT::raw_t)) > 128) ? 2 : 3)
    normtest_accumulate_kernel(const __grid_constant__ StreamParams prm,
                               const __grid_constant__ AccumCarry cy) {
  static_assert(GT::kVec == 4, "four coordinates per thread-row");
  constexpr int V = 4;
  constexpr int H = split_group<GT, false>();
  __shared__ double red[kWarps * 3];
  const int K = prm.K;
  const int tid = threadIdx.x;
  const int chunk = blockIdx.x;
  const bool carry = cy.n_prev > 0.0;
  ChunkGeometry cg = chunk_geometry<GT, kInlineWorkers, false, ADAM>(prm, prm.grads, K, chunk);
  if (carry && ((reinterpret_cast<uintptr_t>(cy.mean_in) + static_cast<uintptr_t>(cg.lo) * 4) & 15))
    cg.aligned = false;
  // does this chunk open its shard?  (the shard: the last s with chunk_prefix[s] <= chunk)
  int lo_s = 0, hi_s = prm.n_shards;
  while (hi_s - lo_s > 1) {
    const int mid = (lo_s + hi_s) >> 1;
    if (prm.chunk_prefix[mid] <= chunk) lo_s = mid; else hi_s = mid;
  }
  const bool opens_shard = chunk == prm.chunk_prefix[lo_s];
  grid_dependency_wait();

  double acc_n2 = 0.0, acc_S = 0.0, acc_Q = 0.0;
  const int64_t hi = cg.hi;
  int64_t row_lo = cg.lo;
  auto vec_ptr = [&](int k, int64_t base) {
    return reinterpret_cast<const typename GT::scalar*>(prm.grads[k]) + base;
  };
  struct State {
    float4 w, m, v;
  };
  auto load_state = [&](int64_t base) {
    State st;
    if (ADAM) {
      st.w = ld_state_16(prm.p + base);
      st.m = ld_state_16(prm.m + base);
      st.v = ld_state_16(prm.v + base);
    }
    return st;
  };
  // the row's new means: written, and (ADAM) consumed by the update of the row's parameters
  auto finish_row = [&](AccumRow<GT>& acc, int64_t base, State& st) {
    float row_n2 = 0.f, row_S = 0.f;
    const float4 mu = acc.finish(cy.inv_total, row_n2, row_S);
    if (prm.gbar) st_stream_16(prm.gbar + base, mu);
    if (ADAM) {
      float2* w2 = reinterpret_cast<float2*>(&st.w);
      float2* m2 = reinterpret_cast<float2*>(&st.m);
      float2* v2 = reinterpret_cast<float2*>(&st.v);
      adamw_pair(prm.adam, prm.adam.omb1, prm.adam.omb2, make_float2(mu.x, mu.y), w2[0], m2[0], v2[0]);
      adamw_pair(prm.adam, prm.adam.omb1, prm.adam.omb2, make_float2(mu.z, mu.w), w2[1], m2[1], v2[1]);
      st_stream_16(prm.p + base, st.w);
      st_stream_16(prm.m + base, st.m);
      st_stream_16(prm.v + base, st.v);
      if (prm.p16) st_bf16x4(prm.p16 + base, st.w);
    }
    acc_n2 += static_cast<double>(row_n2);
    acc_S += static_cast<double>(row_S);
  };

  if constexpr (ROWS > 1) {
    while (cg.aligned && row_lo + static_cast<int64_t>(ROWS) * kThreads * V <= hi) {
      typename GT::raw_t raw[ROWS][KR];
      float4 mo[ROWS];
      State st[ROWS];
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        const int64_t base = row_lo + (static_cast<int64_t>(r) * kThreads + tid) * V;
#pragma unroll
        for (int k = 0; k < KR; ++k)
          if (k < K) raw[r][k] = GT::load_vec(vec_ptr(k, base));
        mo[r] = carry ? ld_state_16(cy.mean_in + base) : make_float4(0.f, 0.f, 0.f, 0.f);
        st[r] = load_state(base);
      }
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        const int64_t base = row_lo + (static_cast<int64_t>(r) * kThreads + tid) * V;
        AccumRow<GT> acc;
        if (carry) acc.init(mo[r]); else acc.init_from(raw[r][0]);
#pragma unroll
        for (int k = 0; k < KR; ++k)
          if (k < K) acc.add(raw[r][k]);
        acc.close_group();
        finish_row(acc, base, st[r]);
      }
      row_lo += static_cast<int64_t>(ROWS) * kThreads * V;
    }
  }

  for (; row_lo < hi; row_lo += kThreads * V) {
    const int64_t base = row_lo + static_cast<int64_t>(tid) * V;
    if (cg.aligned && row_lo + kThreads * V <= hi) {
      AccumRow<GT> acc;
      bool need_centre = !carry;  // uniform across the CTA
      if (carry) acc.init(ld_state_16(cy.mean_in + base));
      State st = load_state(base);  // in flight while the gradients are consumed
      if constexpr (KR > 1) {
        // at most KR workers (the caller's promise for KR > 1): one predicated batch
        typename GT::raw_t raw[KR];
#pragma unroll
        for (int k = 0; k < KR; ++k)
          if (k < K) raw[k] = GT::load_vec(vec_ptr(k, base));
        if (need_centre) acc.init_from(raw[0]);
#pragma unroll
        for (int k = 0; k < KR; ++k)
          if (k < K) acc.add(raw[k]);
      } else {
        // N consecutive workers from k0: all loads first, then the arithmetic
        auto piece = [&](int k0, auto n_tag) {
          constexpr int N = decltype(n_tag)::value;
          typename GT::raw_t raw[N];
#pragma unroll
          for (int k = 0; k < N; ++k) raw[k] = GT::load_vec(vec_ptr(k0 + k, base));
          if (need_centre) {
            acc.init_from(raw[0]);
            need_centre = false;
          }
#pragma unroll
          for (int k = 0; k < N; ++k) acc.add(raw[k]);
        };
        // whole groups of H workers, then the rest in unpredicated pieces of 8, 4, 2, 1
        int k0 = 0;
#pragma unroll 1
        for (; k0 + H <= K; k0 += H) {
          piece(k0, std::integral_constant<int, H>{});
          acc.close_group();
        }
        if (H > 8 && ((K - k0) & 8)) {
          piece(k0, std::integral_constant<int, 8>{});
          k0 += 8;
        }
        if ((K - k0) & 4) {
          piece(k0, std::integral_constant<int, 4>{});
          k0 += 4;
        }
        if ((K - k0) & 2) {
          piece(k0, std::integral_constant<int, 2>{});
          k0 += 2;
        }
        if ((K - k0) & 1) piece(k0, std::integral_constant<int, 1>{});
      }
      acc.close_group();  // adds exact zeros when K is a multiple of H
      finish_row(acc, base, st);
    } else if (base < hi) {
      float sums[2];
      accumulate_scalar_row<GT, ADAM>(prm, cy, K, base, hi, sums);
      acc_n2 += static_cast<double>(sums[0]);
      acc_S += static_cast<double>(sums[1]);
    }
  }
  // the shard's sum so far rides on the first thread's partial of the shard's first chunk
  if (carry && opens_shard && tid == 0)
    acc_S += __ldcg(cy.shard_rec + static_cast<int64_t>(lo_s) * ABS_SHARD_STRIDE + 1);
  CwMax unused;
  unused.init(0);
  write_chunk_record<kStatSums>(prm, chunk, cg.lo, acc_n2, acc_S, acc_Q, unused, red);
}

}  // namespace absnt
