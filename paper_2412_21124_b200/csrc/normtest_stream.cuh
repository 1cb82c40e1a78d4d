// Streaming norm-test kernel (optionally fused with AdamW) and its finalize kernel.
//
// Work decomposition.  Each shard of the flat vector is cut into chunks of
// `chunk_elems` consecutive coordinates (the last chunk of a shard may be short; a
// chunk never straddles a shard boundary).  A CTA processes whole chunks.  Inside a
// chunk, row r assigns the V = 16/sizeof(grad) consecutive coordinates starting at
// chunk_lo + (r*kThreads + tid)*V to thread tid, so the coordinate -> thread -> partial
// sum mapping depends only on (shard offsets, chunk_elems), never on the grid.  One
// {n2, S, Q} triple per chunk goes to scratch; the finalize kernel adds chunk triples in
// a fixed order per shard and shard records in shard order.
//
// Per coordinate (Algorithm 1, "Compute the batch gradient" .. "approximate gradient
// variance"): the K values are summed in fp64 (exact for K <= 32 fp32/bf16 inputs up to
// one final rounding), gbar = fp32(sum/K); deviations g_k - gbar, their squares and g_k^2
// are fp32 over at most V*K terms, then accumulated in fp64.
#pragma once
#include "abs_device.cuh"

namespace absnt {

template <typename GT, int KB, bool EXACT, bool ADAM>
__global__ void __launch_bounds__(kThreads, (KB <= 8 ? 2 : 1))
    normtest_stream_kernel(const __grid_constant__ StreamParams prm) {
  constexpr int V = GT::kVec;
  constexpr int NF4 = V / 4; // float4 per thread-row of an fp32 array
  __shared__ double red[kWarps * 3];

  const int K = EXACT ? KB : prm.K;
  const int tid = threadIdx.x;

  for (int chunk = blockIdx.x; chunk < prm.n_chunks; chunk += gridDim.x) {
    // shard that owns this chunk: largest s with chunk_prefix[s] <= chunk
    int lo_s = 0, hi_s = prm.n_shards;
    while (hi_s - lo_s > 1) {
      const int mid = (lo_s + hi_s) >> 1;
      if (prm.chunk_prefix[mid] <= chunk) lo_s = mid; else hi_s = mid;
    }
    const int64_t lo = prm.shard_off[lo_s] +
                       static_cast<int64_t>(chunk - prm.chunk_prefix[lo_s]) * prm.chunk_elems;
    const int64_t shard_hi = prm.shard_off[lo_s + 1];
    const int64_t hi = (lo + prm.chunk_elems < shard_hi) ? lo + prm.chunk_elems : shard_hi;

    // 16-byte alignment of every stream at this chunk (uniform across the CTA)
    uintptr_t bits = 0;
#pragma unroll
    for (int k = 0; k < KB; ++k)
      if (EXACT || k < K)
        bits |= reinterpret_cast<uintptr_t>(prm.grads[k]) +
                static_cast<uintptr_t>(lo) * sizeof(typename GT::scalar);
    if (prm.gbar) bits |= reinterpret_cast<uintptr_t>(prm.gbar) + static_cast<uintptr_t>(lo) * 4;
    if (ADAM) {
      bits |= reinterpret_cast<uintptr_t>(prm.p) + static_cast<uintptr_t>(lo) * 4;
      bits |= reinterpret_cast<uintptr_t>(prm.m) + static_cast<uintptr_t>(lo) * 4;
      bits |= reinterpret_cast<uintptr_t>(prm.v) + static_cast<uintptr_t>(lo) * 4;
    }
    const bool aligned = (bits & 15) == 0;

    double acc_n2 = 0.0, acc_S = 0.0, acc_Q = 0.0;

    for (int64_t row_lo = lo; row_lo < hi; row_lo += kThreads * V) {
      const int64_t base = row_lo + static_cast<int64_t>(tid) * V;
      const bool fast = aligned && (row_lo + kThreads * V <= hi);

      uint4 raw[KB];
      float pw[V], pm[V], pv[V];
      if (fast) {
#pragma unroll
        for (int k = 0; k < KB; ++k)
          if (EXACT || k < K)
            raw[k] = ld_once_16(reinterpret_cast<const typename GT::scalar*>(prm.grads[k]) + base);
        if (ADAM) {
#pragma unroll
          for (int q = 0; q < NF4; ++q) {
            const float4 a = ld_state_16(prm.p + base + 4 * q);
            const float4 b = ld_state_16(prm.m + base + 4 * q);
            const float4 c = ld_state_16(prm.v + base + 4 * q);
            pw[4 * q + 0] = a.x; pw[4 * q + 1] = a.y; pw[4 * q + 2] = a.z; pw[4 * q + 3] = a.w;
            pm[4 * q + 0] = b.x; pm[4 * q + 1] = b.y; pm[4 * q + 2] = b.z; pm[4 * q + 3] = b.w;
            pv[4 * q + 0] = c.x; pv[4 * q + 1] = c.y; pv[4 * q + 2] = c.z; pv[4 * q + 3] = c.w;
          }
        }
      }

      float gb[V];
      float row_n2 = 0.f, row_S = 0.f, row_Q = 0.f;
#pragma unroll
      for (int e = 0; e < V; ++e) {
        float g[KB];
        if (fast) {
#pragma unroll
          for (int k = 0; k < KB; ++k) g[k] = (EXACT || k < K) ? GT::elem(raw[k], e) : 0.f;
        } else {
          const bool in = base + e < hi;
#pragma unroll
          for (int k = 0; k < KB; ++k)
            g[k] = ((EXACT || k < K) && in) ? GT::load1(prm.grads[k], base + e) : 0.f;
          if (ADAM) {
            pw[e] = in ? prm.p[base + e] : 0.f;
            pm[e] = in ? prm.m[base + e] : 0.f;
            pv[e] = in ? prm.v[base + e] : 0.f;
          }
        }
        double s = 0.0;
#pragma unroll
        for (int k = 0; k < KB; ++k)
          if (EXACT || k < K) s += static_cast<double>(g[k]);
        const float mean = static_cast<float>(s * prm.inv_K);
        float dev2 = 0.f, sq = 0.f;
#pragma unroll
        for (int k = 0; k < KB; ++k)
          if (EXACT || k < K) {
            const float dv = g[k] - mean;
            dev2 = fmaf(dv, dv, dev2);
            sq = fmaf(g[k], g[k], sq);
          }
        gb[e] = mean;
        row_n2 = fmaf(mean, mean, row_n2);
        row_S += dev2;
        row_Q += sq;
        if (ADAM) adamw_elem(prm.adam, mean, pw[e], pm[e], pv[e]);
      }
      acc_n2 += static_cast<double>(row_n2);
      acc_S += static_cast<double>(row_S);
      acc_Q += static_cast<double>(row_Q);

      if (fast) {
#pragma unroll
        for (int q = 0; q < NF4; ++q) {
          if (prm.gbar)
            st_stream_16(prm.gbar + base + 4 * q,
                         make_float4(gb[4 * q], gb[4 * q + 1], gb[4 * q + 2], gb[4 * q + 3]));
          if (ADAM) {
            st_stream_16(prm.p + base + 4 * q,
                         make_float4(pw[4 * q], pw[4 * q + 1], pw[4 * q + 2], pw[4 * q + 3]));
            st_stream_16(prm.m + base + 4 * q,
                         make_float4(pm[4 * q], pm[4 * q + 1], pm[4 * q + 2], pm[4 * q + 3]));
            st_stream_16(prm.v + base + 4 * q,
                         make_float4(pv[4 * q], pv[4 * q + 1], pv[4 * q + 2], pv[4 * q + 3]));
          }
        }
      } else {
#pragma unroll
        for (int e = 0; e < V; ++e) {
          if (base + e < hi) {
            if (prm.gbar) prm.gbar[base + e] = gb[e];
            if (ADAM) {
              prm.p[base + e] = pw[e];
              prm.m[base + e] = pm[e];
              prm.v[base + e] = pv[e];
            }
          }
        }
      }
    }

    block_reduce3<kWarps>(acc_n2, acc_S, acc_Q, red);
    if (tid == 0) {
      double* out = prm.chunk_out + static_cast<int64_t>(chunk) * 4;
      out[0] = acc_n2;
      out[1] = acc_S;
      out[2] = acc_Q;
      out[3] = 0.0;
    }
  }
}

// One CTA.  Per shard: thread t adds chunk triples t, t+1024, ... of that shard in order,
// then a fixed tree over the CTA; thread 0 adds shard records in shard order, takes the
// decision (Algorithm 1: statistic T_k and the If/Else) and writes header + records.
constexpr int kFinalizeThreads = 1024;

__global__ void __launch_bounds__(kFinalizeThreads)
    finalize_kernel(const __grid_constant__ FinalizeParams fp) {
  __shared__ double red[(kFinalizeThreads / 32) * 3];
  double tot_n2 = 0.0, tot_S = 0.0, tot_Q = 0.0;
  for (int s = 0; s < fp.n_shards; ++s) {
    const int c0 = fp.chunk_prefix[s], c1 = fp.chunk_prefix[s + 1];
    double a = 0.0, b = 0.0, c = 0.0;
    for (int ch = c0 + threadIdx.x; ch < c1; ch += kFinalizeThreads) {
      const double2* rec =
          reinterpret_cast<const double2*>(fp.chunk_in + static_cast<int64_t>(ch) * 4);
      const double2 t0 = rec[0], t1 = rec[1];
      a += t0.x;
      b += t0.y;
      c += t1.x;
    }
    block_reduce3<kFinalizeThreads / 32>(a, b, c, red);
    if (threadIdx.x == 0) {
      double* rec = fp.stats + ABS_STATS_HEADER + s * ABS_SHARD_STRIDE;
      rec[0] = a;
      rec[1] = b;
      rec[2] = c;
      rec[3] = 0.0;
      tot_n2 += a;
      tot_S += b;
      tot_Q += c;
    }
  }
  if (threadIdx.x == 0) {
    double T;
    int flags;
    const int64_t b_next = decide_device(tot_S, tot_n2, fp.norm, fp.eta, fp.b_cur, &T, &flags);
    fp.stats[ABS_STAT_N2] = tot_n2;
    fp.stats[ABS_STAT_S] = tot_S;
    fp.stats[ABS_STAT_Q] = tot_Q;
    fp.stats[ABS_STAT_T] = T;
    fp.stats[ABS_STAT_FLAGS] = static_cast<double>(flags);
    fp.stats[ABS_STAT_NORM] = fp.norm;
    fp.stats[ABS_STAT_NCHUNKS] = static_cast<double>(fp.n_chunks);
    fp.stats[7] = 0.0;
    *fp.b_next = b_next;
  }
}

}  // namespace absnt
