// Device-side building blocks shared by the kernels of the norm-test + AdamW library:
// kernel parameter blocks, streaming 128-bit loads/stores, bf16 unpacking, the AdamW
// element update and the fixed-shape fp64 block reduction.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/abs_normtest.h"

namespace absnt {

constexpr int kThreads = 256;  // threads per CTA of the streaming kernels
constexpr int kWarps = kThreads / 32;

// AdamW scalars (Algorithm 1, AdamW lines), prepared on the host in double.
struct AdamScalars {
  float beta1, omb1;  // beta1, 1-beta1
  float beta2, omb2;  // beta2, 1-beta2
  float step_size;    // alpha / (1-beta1^step)
  float inv_bc2;      // 1/(1-beta2^step)
  float eps, decay;   // epsilon, 1-alpha*lambda
};

// Up to kInlineWorkers gradient pointers travel inside the parameter block; calls with more
// workers pass a second kernel parameter, a table of ABS_MAX_WORKERS pointers (8 KB: kernel
// parameters may be up to 32 KB on this architecture), to a kernel of their own, so that the
// common launches keep their small parameter block.
constexpr int kInlineWorkers = 64;
struct WideTable {
  const void* ptrs[ABS_MAX_WORKERS];
};

// Parameter block of the streaming norm-test kernels, passed by value.
struct StreamParams {
  const void* grads[kInlineWorkers];
  int64_t shard_off[ABS_MAX_SHARDS + 1];    // element offsets of the shards
  int32_t chunk_prefix[ABS_MAX_SHARDS + 1]; // first chunk index of each shard
  int64_t d;
  int K;
  int n_shards;
  int n_chunks;
  int chunk_elems; // elements per reduction chunk (a multiple of kThreads*8)
  double inv_K;
  float inv_Kf, neg_Kf;
  float* gbar; // may be null
  float* p;    // fused AdamW only
  float* m;
  float* v;
  uint16_t* p16; // fused AdamW, mixed precision: bf16 copy of the updated parameters, may be null
  // fused AdamW with the gradient clipped by a norm known before the pass (the previous
  // step's ||gbar||^2, read on the device): null = no clipping
  const double* clip_n2;
  double clip_max_norm;
  double* chunk_out; // 4 doubles per chunk: n2, S, Q, 0
  AdamScalars adam;
};

struct FinalizeParams {
  const double* chunk_in;
  int32_t chunk_prefix[ABS_MAX_SHARDS + 1];
  int32_t slice_prefix[ABS_MAX_SHARDS + 1];  // slices of `slice` records before each shard
  int64_t shard_first[ABS_MAX_SHARDS];       // first coordinate of each shard (coordinate-wise test)
  int slice;                                 // records per slice
  int n_shards;
  int n_chunks;
  double* stats; // header + shard records
  int64_t* b_next;
  double eta, norm;
  int64_t b_cur;
};

// ---- programmatic dependent launch ---------------------------------------------------
// Every kernel of the library is launched with the programmatic-stream-serialization
// attribute and executes this wait before its first global-memory access.  The launch
// latency and the index arithmetic of a kernel then overlap the tail of its predecessor
// in the stream, while the wait itself returns only once that predecessor has completed
// and its writes are visible -- so ordering is exactly that of an ordinary launch.
// Without the attribute the instruction is a no-op.
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Lets the next kernel of the stream be scheduled (it was launched with the same attribute)
// once every CTA of this grid has executed this or exited.  The dependent still waits at its
// own grid_dependency_wait for this grid's completion, so only its launch latency and the work
// it does before that wait move forward.
__device__ __forceinline__ void grid_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ---- streaming memory access --------------------------------------------------------
// Gradients are read exactly once and never written: non-coherent path, no L1 allocation.
__device__ __forceinline__ uint4 ld_once_16(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}
// Optimizer state is read once and then overwritten by the same thread.
__device__ __forceinline__ float4 ld_state_16(const float* p) {
  return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream_16(float* p, float4 x) {
  __stcs(reinterpret_cast<float4*>(p), x);
}

// 256-bit accesses (sm_100): with bf16 gradients a thread owns 8 consecutive coordinates,
// i.e. 32 bytes of each fp32 array.  One 256-bit access per array touches whole 32-byte
// sectors; two 128-bit accesses would each touch half of every sector, doubling the
// requests the load/store unit and the L2 see (visible as lg_throttle stalls).
struct alignas(32) Float8 {
  float4 lo, hi;
};
__device__ __forceinline__ Float8 ld_state_32(const float* p) {
  Float8 r;
  asm volatile("ld.global.cs.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r.lo.x), "=f"(r.lo.y), "=f"(r.lo.z), "=f"(r.lo.w), "=f"(r.hi.x),
                 "=f"(r.hi.y), "=f"(r.hi.z), "=f"(r.hi.w)
               : "l"(p));
  return r;
}
__device__ __forceinline__ void st_stream_32(float* p, const float4& lo, const float4& hi) {
  asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(lo.x),
               "f"(lo.y), "f"(lo.z), "f"(lo.w), "f"(hi.x), "f"(hi.y), "f"(hi.z), "f"(hi.w)
               : "memory");
}

// Two fp32 values rounded to nearest-even bf16, `lo` in the low half (the lower address).
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint16_t to_bf16(float x) {
  return static_cast<uint16_t>(pack_bf16x2(x, 0.f) & 0xffffu);
}
// bf16 copy of four / eight consecutive parameters (8- / 16-byte aligned destination)
__device__ __forceinline__ void st_bf16x4(uint16_t* dst, const float4& x) {
  __stcs(reinterpret_cast<uint2*>(dst), make_uint2(pack_bf16x2(x.x, x.y), pack_bf16x2(x.z, x.w)));
}
__device__ __forceinline__ void st_bf16x8(uint16_t* dst, const float4& a, const float4& b) {
  __stcs(reinterpret_cast<uint4*>(dst), make_uint4(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w),
                                                   pack_bf16x2(b.x, b.y), pack_bf16x2(b.z, b.w)));
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// One AdamW coordinate (Algorithm 1: m_k, v_k, the two hats, w_{k+1}):
//   w' = (1-alpha*lambda) w - [alpha/(1-beta1^k)] m' / (sqrt(v'/(1-beta2^k)) + eps).
// The square root and the reciprocal are the hardware approximations (each within
// 2^-22 relative, subnormal operands flushed to zero); they touch only the update term,
// whose magnitude is about alpha, so the result stays orders of magnitude inside the
// 1e-6*max|w| parity tolerance while the step costs 12 instructions instead of ~30
// (measured: 59.6 vs 79.0 thread-instructions per coordinate for the fused K=8 kernel)
// -- this kernel runs at the board's power cap, where instructions saved are bandwidth
// gained.  Flushing only matters for vhat below 1.2e-38 (its root is then below 1.1e-19
// and vanishes against any practical eps).
// omb1, omb2: (1-beta1) and (1-beta2), or those times s and s^2 when the gradient is clipped
// by a scale s known before the pass (GradWeights below) -- clipping then costs no instruction
// per coordinate.
__device__ __forceinline__ void adamw_elem(const AdamScalars& a, float omb1, float omb2, float g,
                                           float& w, float& m, float& v) {
  m = fmaf(a.beta1, m, omb1 * g);
  v = fmaf(a.beta2, v, (omb2 * g) * g);
  float root, inv;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root) : "f"(v * a.inv_bc2));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(root + a.eps));
  w = fmaf(a.decay, w, -((a.step_size * m) * inv));
}

// The same update for two adjacent coordinates with the packed fp32 instructions of sm_100
// (fma/add/mul.f32x2: one issue slot for both lanes, each lane rounded exactly like the
// scalar instruction, so the results are bit-identical to two adamw_elem calls).
__device__ __forceinline__ void adamw_pair(const AdamScalars& a, float omb1, float omb2, float2 g,
                                           float2& w, float2& m, float2& v) {
  const float2 b1 = make_float2(a.beta1, a.beta1), b2 = make_float2(a.beta2, a.beta2);
  m = __ffma2_rn(b1, m, __fmul2_rn(make_float2(omb1, omb1), g));
  v = __ffma2_rn(b2, v, __fmul2_rn(__fmul2_rn(make_float2(omb2, omb2), g), g));
  const float2 vh = __fmul2_rn(v, make_float2(a.inv_bc2, a.inv_bc2));
  float2 root, inv;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root.x) : "f"(vh.x));
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root.y) : "f"(vh.y));
  const float2 den = __fadd2_rn(root, make_float2(a.eps, a.eps));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv.x) : "f"(den.x));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv.y) : "f"(den.y));
  const float2 upd = __fmul2_rn(__fmul2_rn(make_float2(a.step_size, a.step_size), m), inv);
  w = __ffma2_rn(make_float2(a.decay, a.decay), w, make_float2(-upd.x, -upd.y));
}
// The weights (1-beta1), (1-beta2) of the new gradient in the two moments, folded with the
// clipping scale when the call clips by a norm known before the pass:
//   s = min(1, max_norm / (sqrt(n2) + 1e-6));  m' = beta1 m + ((1-beta1) s) g;
//   v' = beta2 v + ((1-beta2) s^2) g^2
// -- AdamW on the clipped gradient s*g.  Without clipping the weights are the plain ones, bit
// for bit.  Read after the dependency wait: n2 is what the previous call's last kernel wrote.
struct GradWeights {
  float omb1, omb2;
};
__device__ __forceinline__ GradWeights grad_weights(const AdamScalars& a, const double* clip_n2,
                                                    double clip_max_norm) {
  GradWeights w{a.omb1, a.omb2};
  if (clip_n2) {
    const double coef = clip_max_norm / (sqrt(__ldcg(clip_n2)) + 1e-6);
    if (coef < 1.0) {
      const float sc = static_cast<float>(coef);
      w.omb1 *= sc;
      w.omb2 *= sc * sc;
    }
  }
  return w;
}

// max(x, +0) that keeps a NaN: the shifted one-pass variance can come out a few ulps below
// zero and is clamped, but a NaN (a non-finite input, or squares that overflowed to inf - inf)
// has to reach the sums so that the call reports ABS_FLAG_NONFINITE.  fmaxf would return 0.
__device__ __forceinline__ float clamp_nonneg(float x) {
  float r;
  asm("max.NaN.f32 %0, %1, 0f00000000;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ double clamp_nonneg(double x) { return x < 0.0 ? 0.0 : x; }

// Mean of K fp32 partial sums: s/K.  For K a power of two the product with 1/K is exact;
// otherwise one residual correction makes K identical inputs return exactly that input.
template <bool POW2>
__device__ __forceinline__ float mean_of_sum(float s, float inv_K, float neg_K) {
  float q = s * inv_K;
  if (!POW2) q = fmaf(fmaf(neg_K, q, s), inv_K, q);
  return q;
}

template <bool POW2>
__device__ __forceinline__ float2 mean_of_sum2(float2 s, float inv_K, float neg_K) {
  const float2 ik = make_float2(inv_K, inv_K);
  float2 q = __fmul2_rn(s, ik);
  if (!POW2) q = __ffma2_rn(__ffma2_rn(make_float2(neg_K, neg_K), q, s), ik, q);
  return q;
}
// Element types of the gradient buffers.
struct F32 {
  static constexpr int kVec = 4; // elements per 16 bytes
  using scalar = float;
  using raw_t = uint4;
  static __device__ __forceinline__ raw_t load_vec(const void* p) { return ld_once_16(p); }
  using sum_t = double; // fp32 addends: only an fp64 sum keeps the mean correctly rounded
  template <bool POW2>
  static __device__ __forceinline__ float mean(double s, const StreamParams& prm) {
    return static_cast<float>(s * prm.inv_K);
  }
  static __device__ __forceinline__ float elem(const uint4& r, int e) {
    return __uint_as_float(e == 0 ? r.x : e == 1 ? r.y : e == 2 ? r.z : r.w);
  }
  // coordinates 2*pi, 2*pi+1 of the vector
  static __device__ __forceinline__ float2 pair(const uint4& r, int pi) {
    return pi == 0 ? make_float2(__uint_as_float(r.x), __uint_as_float(r.y))
                   : make_float2(__uint_as_float(r.z), __uint_as_float(r.w));
  }
  static __device__ __forceinline__ float load1(const void* base, int64_t i) {
    return __ldg(reinterpret_cast<const float*>(base) + i);
  }
};
struct BF16 {
  static constexpr int kVec = 8;
  using scalar = uint16_t;
  using raw_t = uint4;
  static __device__ __forceinline__ raw_t load_vec(const void* p) { return ld_once_16(p); }
  using sum_t = float; // 8-bit significands: fp32 partial sums are exact within 13 binades
  template <bool POW2>
  static __device__ __forceinline__ float mean(float s, const StreamParams& prm) {
    return mean_of_sum<POW2>(s, prm.inv_Kf, prm.neg_Kf);
  }
  static __device__ __forceinline__ float elem(const uint4& r, int e) {
    const uint32_t w = (e >> 1) == 0 ? r.x : (e >> 1) == 1 ? r.y : (e >> 1) == 2 ? r.z : r.w;
    return (e & 1) ? bf16_hi(w) : bf16_lo(w);
  }
  static __device__ __forceinline__ float2 pair(const uint4& r, int pi) {
    const uint32_t w = pi == 0 ? r.x : pi == 1 ? r.y : pi == 2 ? r.z : r.w;
    return make_float2(bf16_lo(w), bf16_hi(w));
  }
  static __device__ __forceinline__ float load1(const void* base, int64_t i) {
    return __uint_as_float(
        static_cast<uint32_t>(__ldg(reinterpret_cast<const uint16_t*>(base) + i)) << 16);
  }
};
// bf16 gradients taken four coordinates (8 bytes) per thread-row instead of eight: half the
// registers per worker, so that the K=32 kernels keep two CTAs per SM resident.
struct BF16H {
  static constexpr int kVec = 4;
  using scalar = uint16_t;
  using raw_t = uint2;
  using sum_t = float;
  static __device__ __forceinline__ raw_t load_vec(const void* p) {
    uint2 r;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
    return r;
  }
  template <bool POW2>
  static __device__ __forceinline__ float mean(float s, const StreamParams& prm) {
    return mean_of_sum<POW2>(s, prm.inv_Kf, prm.neg_Kf);
  }
  static __device__ __forceinline__ float elem(const uint2& r, int e) {
    const uint32_t w = (e >> 1) ? r.y : r.x;
    return (e & 1) ? bf16_hi(w) : bf16_lo(w);
  }
  static __device__ __forceinline__ float2 pair(const uint2& r, int pi) {
    const uint32_t w = pi ? r.y : r.x;
    return make_float2(bf16_lo(w), bf16_hi(w));
  }
  static __device__ __forceinline__ float load1(const void* base, int64_t i) {
    return BF16::load1(base, i);
  }
};

// Fixed-shape reduction of three doubles over a CTA of NW warps.  Every call adds the
// same operands in the same order, so the result is independent of scheduling.
// Result valid in thread 0.  `sm` holds NW*3 doubles.
template <int NW>
__device__ __forceinline__ void block_reduce3(double& a, double& b, double& c, double* sm) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    a += __shfl_down_sync(0xffffffffu, a, off);
    b += __shfl_down_sync(0xffffffffu, b, off);
    c += __shfl_down_sync(0xffffffffu, c, off);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    sm[warp * 3 + 0] = a;
    sm[warp * 3 + 1] = b;
    sm[warp * 3 + 2] = c;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double ra = sm[0], rb = sm[1], rc = sm[2];
#pragma unroll
    for (int w = 1; w < NW; ++w) {
      ra += sm[w * 3 + 0];
      rb += sm[w * 3 + 1];
      rc += sm[w * 3 + 2];
    }
    a = ra;
    b = rb;
    c = rc;
  }
  __syncthreads();
}

// The decision, device side (same expression order as the host's abs_decide).
__device__ __forceinline__ int64_t decide_device(double S, double n2, double norm, double eta,
                                                 int64_t b_cur, double* T_out, int* flags_out) {
  int flags = 0;
  const double T = (S / norm) / ((eta * eta) * n2);
  int64_t b_next = b_cur;
  if (!isfinite(S) || !isfinite(n2)) {
    flags |= ABS_FLAG_NONFINITE;
  } else {
    if (n2 == 0.0) flags |= ABS_FLAG_DEGENERATE;
    if (T > static_cast<double>(b_cur)) {
      flags |= ABS_FLAG_VIOLATED;
      b_next = (T >= 4611686018427387904.0) ? INT64_MAX : static_cast<int64_t>(ceil(T));
    }
  }
  *T_out = T;
  *flags_out = flags;
  return b_next;
}

}  // namespace absnt
