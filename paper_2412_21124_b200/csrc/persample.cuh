// Per-sample form of the norm test (Eq. 3 with the Var definition before it): column
// mean and column sum of squared deviations of a row-major [b, ld] matrix whose rows
// are per-sample gradients, reading the matrix once.
//
// Pass 1 (2-D grid: column block x row block): a thread owns VC adjacent columns and
// walks its row block in groups of kGroup rows.  Each value is consumed once, as it arrives:
// per group and column the thread accumulates sum(x) in fp64 and, about a centre c close to
// the column mean (the first row for the first group, the running mean afterwards),
// sum((x-c)^2) in fp32; then
//     mu_g = sum(x)/n_g,   M2_g = sum((x-c)^2) - n_g (mu_g-c)^2        (shift identity)
// and the group is merged into the running {mean, M2} with the pairwise update
//     delta = mu_g - mean;  mean += delta*n_g/(n+n_g);  M2 += M2_g + delta^2*n*n_g/(n+n_g)
// (law of total variance).  Because no value is needed twice, the rows are loaded in half
// groups, the next half in flight while the current one is consumed.  It writes
// {mean, M2, Q} per (row block, column).
// Pass 2 (one thread per column): merges the row blocks in index order with the same
// update, writes gbar, and reduces {gbar^2, M2, Q} over 128-column chunks for the
// shared finalize kernel.
// Also here: the stand-alone AdamW kernel.
#pragma once
#include "abs_device.cuh"

namespace absnt {

constexpr int kGroup = 16;      // rows per group (one shift centre, one merge)
constexpr int kHalf = kGroup / 2; // rows per load batch
constexpr int kPsThreads = 128; // threads per CTA of the per-sample kernels

struct PersampleParams {
  const float* G;
  int64_t b, d, ld;
  int rows_per_block;
  int n_row_blocks;
  double* ws_mean; // [n_row_blocks][d]
  double* ws_m2;
  double* ws_q;
  float* gbar;
  double* chunk_out; // 4 doubles per kPsThreads-column chunk
};

// rows r .. r+kHalf-1 of this thread's columns; rows at or past r_end read as zero
template <int VC, bool FULL>
__device__ __forceinline__ void ps_load_half(const PersampleParams& prm, int64_t r, int64_t r_end,
                                             int64_t c0, bool vec_cols, float (&x)[kHalf][VC]) {
#pragma unroll
  for (int j = 0; j < kHalf; ++j) {
    const float* row = prm.G + (r + j) * prm.ld + c0;
    if (FULL || r + j < r_end) {
      if (VC == 4 && vec_cols) {
        const uint4 t = ld_once_16(row);
        x[j][0] = __uint_as_float(t.x);
        x[j][1 % VC] = __uint_as_float(t.y);
        x[j][2 % VC] = __uint_as_float(t.z);
        x[j][3 % VC] = __uint_as_float(t.w);
      } else {
#pragma unroll
        for (int i = 0; i < VC; ++i) x[j][i] = (c0 + i < prm.d) ? __ldg(row + i) : 0.f;
      }
    } else {
#pragma unroll
      for (int i = 0; i < VC; ++i) x[j][i] = 0.f;
    }
  }
}

// Accumulators of one group: sum(x) in two fp64 chains (even and odd rows), the shifted
// squares and the plain squares in fp32.
template <int VC>
struct PsGroup {
  double s0[VC], s1[VC];
  float c[VC], s2[VC], q[VC];
};

template <int VC, bool FULL>
__device__ __forceinline__ void ps_consume_half(PsGroup<VC>& g, const float (&x)[kHalf][VC],
                                                int n_live) {
#pragma unroll
  for (int j = 0; j < kHalf; ++j) {
    if (FULL || j < n_live) {
#pragma unroll
      for (int i = 0; i < VC; ++i) {
        const float v = x[j][i];
        if (j & 1) g.s1[i] += static_cast<double>(v); else g.s0[i] += static_cast<double>(v);
        const float dv = v - g.c[i];
        g.s2[i] = fmaf(dv, dv, g.s2[i]);
        g.q[i] = fmaf(v, v, g.q[i]);
      }
    }
  }
}

template <int VC>
__global__ void __launch_bounds__(kPsThreads, 3)
    persample_partial_kernel(const __grid_constant__ PersampleParams prm) {
  const int64_t c0 = (static_cast<int64_t>(blockIdx.x) * kPsThreads + threadIdx.x) * VC;
  grid_dependency_wait();
  if (c0 >= prm.d) return;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * prm.rows_per_block;
  const int64_t r1 = (r0 + prm.rows_per_block < prm.b) ? r0 + prm.rows_per_block : prm.b;
  const bool vec_cols = (c0 + VC <= prm.d);

  double mean[VC], m2[VC], qq[VC];
#pragma unroll
  for (int i = 0; i < VC; ++i) mean[i] = m2[i] = qq[i] = 0.0;
  int64_t n = 0;
  PsGroup<VC> g;
  float xa[kHalf][VC], xb[kHalf][VC];

  // centre of the next group and cleared accumulators; `first` = first row of the group
  auto open_group = [&](const float (&first)[VC]) {
#pragma unroll
    for (int i = 0; i < VC; ++i) {
      g.c[i] = (n == 0) ? first[i] : static_cast<float>(mean[i]);
      g.s0[i] = g.s1[i] = 0.0;
      g.s2[i] = g.q[i] = 0.f;
    }
  };
  auto close_group = [&](int ng) {
    const double dn = static_cast<double>(ng);
    const double nn = static_cast<double>(n + ng);
    const double w_mean = dn / nn;
    const double w_m2 = static_cast<double>(n) * w_mean;
#pragma unroll
    for (int i = 0; i < VC; ++i) {
      const double sum = g.s0[i] + g.s1[i];
      // a power-of-two count divides exactly by multiplication; a ragged count by division,
      // so that identical rows give their common value exactly
      const double mu = (ng == kGroup) ? sum * (1.0 / kGroup) : sum / dn;
      const double dc = mu - static_cast<double>(g.c[i]);
      const double m2g = clamp_nonneg(static_cast<double>(g.s2[i]) - dn * dc * dc);
      const double delta = mu - mean[i];
      mean[i] += delta * w_mean;
      m2[i] += m2g + delta * delta * w_m2;
      qq[i] += static_cast<double>(g.q[i]);
    }
    n += ng;
  };

  const int64_t n_full = (r1 - r0) / kGroup;
  int64_t r = r0;
  if (n_full > 0) ps_load_half<VC, true>(prm, r, r1, c0, vec_cols, xa);
  for (int64_t gi = 0; gi < n_full; ++gi) {
    open_group(xa[0]);
    ps_load_half<VC, true>(prm, r + kHalf, r1, c0, vec_cols, xb);
    ps_consume_half<VC, true>(g, xa, kHalf);
    if (gi + 1 < n_full) ps_load_half<VC, true>(prm, r + kGroup, r1, c0, vec_cols, xa);
    ps_consume_half<VC, true>(g, xb, kHalf);
    close_group(kGroup);
    r += kGroup;
  }
  if (r < r1) {  // the last, ragged group of the row block
    const int ng = static_cast<int>(r1 - r);
    ps_load_half<VC, false>(prm, r, r1, c0, vec_cols, xa);
    ps_load_half<VC, false>(prm, r + kHalf, r1, c0, vec_cols, xb);
    open_group(xa[0]);
    ps_consume_half<VC, false>(g, xa, ng);
    ps_consume_half<VC, false>(g, xb, ng - kHalf);
    close_group(ng);
  }
  const int64_t o = static_cast<int64_t>(blockIdx.y) * prm.d + c0;
#pragma unroll
  for (int i = 0; i < VC; ++i) {
    if (c0 + i < prm.d) {
      prm.ws_mean[o + i] = mean[i];
      prm.ws_m2[o + i] = m2[i];
      prm.ws_q[o + i] = qq[i];
    }
  }
}

__global__ void __launch_bounds__(kPsThreads)
    persample_merge_kernel(const __grid_constant__ PersampleParams prm) {
  __shared__ double red[(kPsThreads / 32) * 3];
  const int64_t c = static_cast<int64_t>(blockIdx.x) * kPsThreads + threadIdx.x;
  grid_dependency_wait();
  double a = 0.0, s = 0.0, q = 0.0;
  if (c < prm.d) {
    double mean = 0.0, m2 = 0.0;
    int64_t n = 0;
    // row blocks in index order, eight records in flight at a time
    for (int rb0 = 0; rb0 < prm.n_row_blocks; rb0 += 8) {
      double mu[8], mm[8], qq[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int rb = rb0 + u;
        const bool in = rb < prm.n_row_blocks;
        const int64_t o = static_cast<int64_t>(in ? rb : 0) * prm.d + c;
        mu[u] = in ? prm.ws_mean[o] : 0.0;
        mm[u] = in ? prm.ws_m2[o] : 0.0;
        qq[u] = in ? prm.ws_q[o] : 0.0;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int rb = rb0 + u;
        if (rb < prm.n_row_blocks) {
          const int64_t r0 = static_cast<int64_t>(rb) * prm.rows_per_block;
          const int64_t nb = (r0 + prm.rows_per_block < prm.b) ? prm.rows_per_block : prm.b - r0;
          const double nn = static_cast<double>(n + nb);
          const double w_mean = static_cast<double>(nb) / nn;
          const double delta = mu[u] - mean;
          mean += delta * w_mean;
          m2 += mm[u] + delta * delta * (static_cast<double>(n) * w_mean);
          q += qq[u];
          n += nb;
        }
      }
    }
    const float gb = static_cast<float>(mean);
    prm.gbar[c] = gb;
    a = static_cast<double>(gb) * static_cast<double>(gb);
    s = m2;
  }
  block_reduce3<kPsThreads / 32>(a, s, q, red);
  if (threadIdx.x == 0) {
    double* out = prm.chunk_out + static_cast<int64_t>(blockIdx.x) * 4;
    out[0] = a;
    out[1] = s;
    out[2] = q;
    out[3] = 0.0;
  }
}

// Stand-alone AdamW (Algorithm 1, AdamW lines), in place.  With `n2_dev` non-null the
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
  float scale = 1.f;
  if (n2_dev) {
    const double coef = max_norm / (sqrt(*n2_dev) + 1e-6);
    scale = coef < 1.0 ? static_cast<float>(coef) : 1.f;
  }
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
      adamw_elem(a, scale * g0.x, p0.x, m0.x, v0.x);
      adamw_elem(a, scale * g0.y, p0.y, m0.y, v0.y);
      adamw_elem(a, scale * g0.z, p0.z, m0.z, v0.z);
      adamw_elem(a, scale * g0.w, p0.w, m0.w, v0.w);
      st_stream_16(p + 4 * i, p0);
      st_stream_16(m + 4 * i, m0);
      st_stream_16(v + 4 * i, v0);
      if (p16) st_bf16x4(p16 + 4 * i, p0);
      adamw_elem(a, scale * g1.x, p1.x, m1.x, v1.x);
      adamw_elem(a, scale * g1.y, p1.y, m1.y, v1.y);
      adamw_elem(a, scale * g1.z, p1.z, m1.z, v1.z);
      adamw_elem(a, scale * g1.w, p1.w, m1.w, v1.w);
      st_stream_16(p + 4 * j, p1);
      st_stream_16(m + 4 * j, m1);
      st_stream_16(v + 4 * j, v1);
      if (p16) st_bf16x4(p16 + 4 * j, p1);
    }
    if (i < nvec) {
      const float4 gg = __ldcs(reinterpret_cast<const float4*>(g) + i);
      float4 pp = ld_state_16(p + 4 * i), mm = ld_state_16(m + 4 * i), vv = ld_state_16(v + 4 * i);
      adamw_elem(a, scale * gg.x, pp.x, mm.x, vv.x);
      adamw_elem(a, scale * gg.y, pp.y, mm.y, vv.y);
      adamw_elem(a, scale * gg.z, pp.z, mm.z, vv.z);
      adamw_elem(a, scale * gg.w, pp.w, mm.w, vv.w);
      st_stream_16(p + 4 * i, pp);
      st_stream_16(m + 4 * i, mm);
      st_stream_16(v + 4 * i, vv);
      if (p16) st_bf16x4(p16 + 4 * i, pp);
    }
    // tail (d % 4 elements) by the first threads of block 0
    const int64_t t = (nvec << 2) + threadIdx.x;
    if (blockIdx.x == 0 && t < d) {
      float pp = p[t], mm = m[t], vv = v[t];
      adamw_elem(a, scale * g[t], pp, mm, vv);
      p[t] = pp;
      m[t] = mm;
      v[t] = vv;
      if (p16) p16[t] = to_bf16(pp);
    }
  } else {
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < d;
         i += stride) {
      float pp = p[i], mm = m[i], vv = v[i];
      adamw_elem(a, scale * g[i], pp, mm, vv);
      p[i] = pp;
      m[i] = mm;
      v[i] = vv;
      if (p16) p16[i] = to_bf16(pp);
    }
  }
}

}  // namespace absnt
