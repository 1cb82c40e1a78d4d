// C ABI of the norm-test + AdamW library: argument validation, launch configuration and
// the host-side helpers.  Every step of the path runs in the kernels; this file only
// checks, sizes and launches.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <unordered_map>
#include <utility>

#include "launch.cuh"
#include "normtest_accumulate.cuh"
#include "persample.cuh"

using namespace absnt;

// The kernels behind these are instantiated in stream_inst.cu, once per combination.
namespace absnt {
#define ABS_DECLARE_STREAM(GT, ADAM, STAT) \
  extern template cudaError_t launch_stream<GT, ADAM, STAT>(const StreamParams&, const WideTable*, \
                                                            cudaStream_t);
ABS_DECLARE_STREAM(F32, true, kStatSums)
ABS_DECLARE_STREAM(BF16, true, kStatSums)
ABS_DECLARE_STREAM(F32, false, kStatSumsQ)
ABS_DECLARE_STREAM(BF16, false, kStatSumsQ)
ABS_DECLARE_STREAM(F32, false, kStatSums)
ABS_DECLARE_STREAM(BF16, false, kStatSums)
ABS_DECLARE_STREAM(F32, true, kStatCoordwise)
ABS_DECLARE_STREAM(BF16, true, kStatCoordwise)
ABS_DECLARE_STREAM(F32, false, kStatCoordwise)
ABS_DECLARE_STREAM(BF16, false, kStatCoordwise)
#undef ABS_DECLARE_STREAM
}  // namespace absnt

namespace {

thread_local int g_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return ABS_ERR_CUDA;
}

// Elements per reduction chunk (= the work of one CTA).  A function of the problem (d and
// the entry point) alone, so that the summation tree -- and with it every output bit --
// never depends on the launch.  Measured at d=124M: the fused kernels like 8192 (+0.5..2%
// over 16384; 4096 costs the staged kernel 4% in pipeline fill and drain); the unfused
// test, bound by instruction issue, likes 16384 (the per-chunk reduction costs it 2.5% at
// 8192).  abs_stats_bytes sizes the scratch for the smaller of the two.
int chunk_elems_for(int64_t d, bool fused) {
  return d >= (int64_t{1} << 23) ? (fused ? 8192 : 16384) : 4096;
}

bool finite_nonneg(float x) { return std::isfinite(x) && x >= 0.f; }

int check_hparams(const abs_adamw_hparams* h, int64_t step) {
  if (!h) return ABS_ERR_NULL;
  if (step < 1) return ABS_ERR_RANGE;
  if (!finite_nonneg(h->lr) || !finite_nonneg(h->eps) || !finite_nonneg(h->weight_decay))
    return ABS_ERR_RANGE;
  if (!(h->beta1 >= 0.f && h->beta1 < 1.f) || !(h->beta2 >= 0.f && h->beta2 < 1.f))
    return ABS_ERR_RANGE;
  return ABS_OK;
}

AdamScalars make_adam(const abs_adamw_hparams* h, int64_t step) {
  AdamScalars a;
  const double b1 = h->beta1, b2 = h->beta2;
  a.beta1 = h->beta1;
  a.omb1 = static_cast<float>(1.0 - b1);
  a.beta2 = h->beta2;
  a.omb2 = static_cast<float>(1.0 - b2);
  a.step_size = static_cast<float>(static_cast<double>(h->lr) /
                                   (1.0 - std::pow(b1, static_cast<double>(step))));
  a.inv_bc2 = static_cast<float>(1.0 / (1.0 - std::pow(b2, static_cast<double>(step))));
  a.eps = h->eps;
  a.decay =
      static_cast<float>(1.0 - static_cast<double>(h->lr) * static_cast<double>(h->weight_decay));
  return a;
}

// Largest cluster (8, 4, 2 or 1 CTAs) of finalize_kernel that the current device can
// co-schedule (asked for the variant with the larger shared-memory footprint), asked once per
// device and cached.  A refusal (SM partitioning, a shared
// device) or a failing query means 1: a plain single-CTA launch, which cannot be refused for
// lack of co-scheduling.  The sums do not depend on the cluster size, so the fallback changes
// no output bit.
int finalize_max_cluster() {
  static std::mutex mu;
  static int cached[64] = {};  // 0 = not asked yet
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev]) return cached[dev];
  }
  int best = 1;
  for (int n = kFinalizeMaxCtas; n > 1; n /= 2) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n);
    cfg.blockDim = dim3(kFinalizeThreads);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = n;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int active = 0;
    if (cudaOccupancyMaxActiveClusters(&active, finalize_kernel<true>, &cfg) == cudaSuccess &&
        active >= 1) {
      best = n;
      break;
    }
  }
  (void)cudaGetLastError();  // a refused query is an answer, not an error of the call
  std::lock_guard<std::mutex> lock(mu);
  cached[dev] = best;
  return best;
}

// The finalize kernel runs as one thread-block cluster.  The slice size (and with it the
// shape of every sum) follows from the chunk counts alone; the cluster size only decides how
// many warps share the slices.  `max_ctas` is finalize_max_cluster(), queried by the caller
// before its first launch so that nothing that can be foreseen fails after it.
cudaError_t launch_finalize(FinalizeParams fp, int max_ctas, cudaStream_t st,
                            bool coordwise = false) {
  int slice = kFinalizeSlice;
  for (;;) {
    int64_t n = 0;
    for (int s = 0; s < fp.n_shards; ++s)
      n += (fp.chunk_prefix[s + 1] - fp.chunk_prefix[s] + slice - 1) / slice;
    if (n <= kFinalizeMaxSlices) break;
    slice *= 2;
  }
  fp.slice = slice;
  fp.slice_prefix[0] = 0;
  for (int s = 0; s < fp.n_shards; ++s)
    fp.slice_prefix[s + 1] =
        fp.slice_prefix[s] + (fp.chunk_prefix[s + 1] - fp.chunk_prefix[s] + slice - 1) / slice;
  const int n_slices = fp.slice_prefix[fp.n_shards];
  unsigned n_ctas = 1;
  while (static_cast<int>(n_ctas) < max_ctas &&
         static_cast<int>(n_ctas) * kFinalizeSlicesPerCta < n_slices)
    n_ctas *= 2;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_ctas);
  cfg.blockDim = dim3(kFinalizeThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = n_ctas;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = n_ctas > 1 ? 2 : 1;  // one CTA: an ordinary launch (its own implicit cluster)
  return coordwise ? cudaLaunchKernelEx(&cfg, finalize_kernel<true>, fp)
                   : cudaLaunchKernelEx(&cfg, finalize_kernel<false>, fp);
}

bool misaligned(const void* p, size_t a) {
  return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0;
}

// [a, a+na) and [b, b+nb) share a byte
bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
  return a0 < b0 + nb && b0 < a0 + na;
}

// Aliasing rule of the norm-test calls: no output range may share a byte with a gradient
// buffer or with another output (the kernels read every input coordinate exactly once and
// give no ordering between a chunk's reads and another chunk's writes).
struct Range {
  const void* p;
  size_t bytes;
};
bool any_alias(const void* const* grads, int K, size_t grad_bytes, const Range* outs, int n_outs) {
  for (int i = 0; i < n_outs; ++i) {
    if (!outs[i].p) continue;
    for (int k = 0; k < K; ++k)
      if (overlaps(outs[i].p, outs[i].bytes, grads[k], grad_bytes)) return true;
    for (int j = i + 1; j < n_outs; ++j)
      if (outs[j].p && overlaps(outs[i].p, outs[i].bytes, outs[j].p, outs[j].bytes)) return true;
  }
  return false;
}

struct Layout {
  int n_shards;
  int n_chunks;
  int chunk_elems;
  int64_t shard_off[ABS_MAX_SHARDS + 1];
  int32_t chunk_prefix[ABS_MAX_SHARDS + 1];
};

// Validates the shard table and cuts the shards into chunks.
int make_layout(int64_t d, const int64_t* shard_offsets, int n_shards, bool fused, Layout* L) {
  if (!shard_offsets) n_shards = 1;
  if (n_shards < 1 || n_shards > ABS_MAX_SHARDS) return ABS_ERR_RANGE;
  L->n_shards = n_shards;
  L->chunk_elems = chunk_elems_for(d, fused);
  if (!shard_offsets) {
    L->shard_off[0] = 0;
    L->shard_off[1] = d;
  } else {
    if (shard_offsets[0] != 0 || shard_offsets[n_shards] != d) return ABS_ERR_SHARDS;
    for (int s = 0; s < n_shards; ++s)
      if (shard_offsets[s + 1] < shard_offsets[s]) return ABS_ERR_SHARDS;
    std::memcpy(L->shard_off, shard_offsets, sizeof(int64_t) * (n_shards + 1));
  }
  int64_t chunks = 0;
  for (int s = 0; s < n_shards; ++s) {
    L->chunk_prefix[s] = static_cast<int32_t>(chunks);
    chunks += (L->shard_off[s + 1] - L->shard_off[s] + L->chunk_elems - 1) / L->chunk_elems;
    if (chunks > INT32_MAX) return ABS_ERR_RANGE;
  }
  L->chunk_prefix[n_shards] = static_cast<int32_t>(chunks);
  L->n_chunks = static_cast<int>(chunks);
  return ABS_OK;
}

// A wait of the staged kernels' kind on a barrier that nothing will ever complete: one thread
// polls `polls` times with the same instruction as mbar_wait_bounded and reports that it gave
// up and how long that took.  Nothing here can hang: the loop has a fixed trip count.
__global__ void bounded_wait_selftest_kernel(int polls, long long* out) {
  __shared__ uint64_t bar;
  grid_dependency_wait();
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    bool completed = false;
    for (int i = 0; i < polls && !completed; ++i) completed = mbar_try_wait(&bar, 0u);
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    out[0] = completed ? 0 : 1;
    out[1] = t1 - t0;
  }
}

// ---------------------------------------------------------------------------------------
// abs_normtest_adamw_noalloc: the fused step with its chunk records in an array that is
// part of the library image, for callers that cannot allocate device memory.
// ---------------------------------------------------------------------------------------
// One {n2, S, Q, 0} record per chunk.  Lives in every device's copy of the module.
static __device__ __align__(256) double g_noalloc_chunk_records[ABS_NOALLOC_MAX_CHUNKS * 4];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
double* g_noalloc_device_ptr[kMaxDevices] = {};  // device address of the array, per device

// In host code `g_noalloc_chunk_records` is only a handle for the runtime, not an address
// a kernel could use: the device address is looked up once per device (with that device
// current) and cached.
int noalloc_records_for_current_device(double** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= kMaxDevices) return ABS_ERR_RANGE;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_device_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_chunk_records);
    if (e != cudaSuccess) return cuda_fail(e);
    g_noalloc_device_ptr[dev] = static_cast<double*>(p);
  }
  *out = g_noalloc_device_ptr[dev];
  return ABS_OK;
}

// The one body behind abs_norm_test, abs_normtest_adamw(_mixed) and the no-alloc variant.
// `builtin_records`: the per-chunk records go to the array built into the library (no-alloc
// variant; stats_out is then header + shard records only) instead of the tail of stats_out.
int run_norm_test(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                  const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                  void* stats_out, float* gbar_out, int64_t* b_next_out, float* params, float* m,
                  float* v, void* params_bf16, const abs_adamw_hparams* hparams, int64_t step,
                  bool fused, abs_stream_t stream, bool builtin_records = false,
                  int stat = -1, const double* clip_n2 = nullptr, double clip_max_norm = 0.0) {
  if (stat < 0) stat = kStatSums;
  if (!grads || !stats_out || !b_next_out) return ABS_ERR_NULL;
  if (!fused && !gbar_out) return ABS_ERR_NULL;
  if (fused && (!params || !m || !v)) return ABS_ERR_NULL;
  if (dtype != ABS_F32 && dtype != ABS_BF16) return ABS_ERR_DTYPE;
  if (K < 1 || K > ABS_MAX_WORKERS || d < 1 || b_cur < 1) return ABS_ERR_RANGE;
  if (!std::isfinite(eta) || !(eta > 0.0)) return ABS_ERR_RANGE;
  if (fused) {
    const int rc = check_hparams(hparams, step);
    if (rc != ABS_OK) return rc;
  }
  const size_t esz = (dtype == ABS_F32) ? 4 : 2;
  for (int k = 0; k < K; ++k) {
    if (!grads[k]) return ABS_ERR_NULL;
    if (misaligned(grads[k], esz)) return ABS_ERR_ALIGN;
  }
  if (misaligned(stats_out, 16) || misaligned(b_next_out, 8)) return ABS_ERR_ALIGN;
  if (gbar_out && misaligned(gbar_out, 4)) return ABS_ERR_ALIGN;
  if (fused && (misaligned(params, 4) || misaligned(m, 4) || misaligned(v, 4)))
    return ABS_ERR_ALIGN;
  if (params_bf16 && misaligned(params_bf16, 2)) return ABS_ERR_ALIGN;

  Layout L;
  const int rc = make_layout(d, shard_offsets, n_shards, fused, &L);
  if (rc != ABS_OK) return rc;
  if (builtin_records && L.n_chunks > ABS_NOALLOC_MAX_CHUNKS) return ABS_ERR_TOO_LARGE;

  const size_t ud = static_cast<size_t>(d);
  const size_t stats_bytes =
      builtin_records
          ? sizeof(double) * (ABS_STATS_HEADER + static_cast<size_t>(L.n_shards) * ABS_SHARD_STRIDE)
          : abs_stats_bytes(d, L.n_shards);
  const Range outs[] = {{gbar_out, ud * 4}, {params, ud * 4},       {m, ud * 4},
                        {v, ud * 4},        {params_bf16, ud * 2},  {stats_out, stats_bytes},
                        {b_next_out, 8}};
  if (any_alias(grads, K, ud * esz, outs, 7)) return ABS_ERR_ALIAS;

  // everything that can be refused is asked before the first launch
  const int finalize_ctas = finalize_max_cluster();
  double* stats = static_cast<double*>(stats_out);
  double* chunk_out =
      stats + ABS_STATS_HEADER + static_cast<size_t>(L.n_shards) * ABS_SHARD_STRIDE;
  if (builtin_records) {
    // every record the final reduction reads is written by this call's first kernel, so the
    // previous call's contents of the shared array are never observed
    const int rc2 = noalloc_records_for_current_device(&chunk_out);
    if (rc2 != ABS_OK) return rc2;
  }

  StreamParams prm;
  std::memset(&prm, 0, sizeof prm);
  WideTable wide_table;  // only filled and passed for more than kInlineWorkers workers
  const WideTable* wide = nullptr;
  if (K <= kInlineWorkers) {
    for (int k = 0; k < K; ++k) prm.grads[k] = grads[k];
  } else {
    for (int k = 0; k < K; ++k) wide_table.ptrs[k] = grads[k];
    for (int k = K; k < ABS_MAX_WORKERS; ++k) wide_table.ptrs[k] = nullptr;
    wide = &wide_table;
  }
  std::memcpy(prm.shard_off, L.shard_off, sizeof(int64_t) * (L.n_shards + 1));
  std::memcpy(prm.chunk_prefix, L.chunk_prefix, sizeof(int32_t) * (L.n_shards + 1));
  prm.d = d;
  prm.K = K;
  prm.n_shards = L.n_shards;
  prm.n_chunks = L.n_chunks;
  prm.chunk_elems = L.chunk_elems;
  prm.inv_K = 1.0 / static_cast<double>(K);
  prm.inv_Kf = static_cast<float>(prm.inv_K);
  prm.neg_Kf = -static_cast<float>(K);
  prm.gbar = gbar_out;
  prm.p = params;
  prm.m = m;
  prm.v = v;
  prm.p16 = static_cast<uint16_t*>(params_bf16);
  prm.chunk_out = chunk_out;
  prm.clip_n2 = clip_n2;
  prm.clip_max_norm = clip_max_norm;
  if (fused) prm.adam = make_adam(hparams, step);

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  const bool f32 = dtype == ABS_F32;
  if (stat == kStatCoordwise) {
    e = fused ? (f32 ? launch_stream<F32, true, kStatCoordwise>(prm, wide, st)
                     : launch_stream<BF16, true, kStatCoordwise>(prm, wide, st))
              : (f32 ? launch_stream<F32, false, kStatCoordwise>(prm, wide, st)
                     : launch_stream<BF16, false, kStatCoordwise>(prm, wide, st));
  } else if (fused) {
    e = f32 ? launch_stream<F32, true, kStatSums>(prm, wide, st)
            : launch_stream<BF16, true, kStatSums>(prm, wide, st);
  } else if (stat == kStatSumsQ) {
    e = f32 ? launch_stream<F32, false, kStatSumsQ>(prm, wide, st)
            : launch_stream<BF16, false, kStatSumsQ>(prm, wide, st);
  } else {
    e = f32 ? launch_stream<F32, false, kStatSums>(prm, wide, st)
            : launch_stream<BF16, false, kStatSums>(prm, wide, st);
  }
  if (e != cudaSuccess) return cuda_fail(e);

  FinalizeParams fp;
  std::memset(&fp, 0, sizeof fp);
  fp.chunk_in = chunk_out;
  std::memcpy(fp.chunk_prefix, L.chunk_prefix, sizeof(int32_t) * (L.n_shards + 1));
  fp.n_shards = L.n_shards;
  fp.n_chunks = L.n_chunks;
  fp.stats = stats;
  fp.b_next = b_next_out;
  fp.eta = eta;
  fp.norm = static_cast<double>(K);
  fp.b_cur = b_cur;
  std::memcpy(fp.shard_first, L.shard_off, sizeof(int64_t) * L.n_shards);
  e = launch_finalize(fp, finalize_ctas, st, stat == kStatCoordwise);
  if (e != cudaSuccess) return cuda_fail(e);
  return ABS_OK;
}

// The one body behind abs_norm_test_accumulate and its closing form with AdamW.
int run_accumulate(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                   const int64_t* shard_offsets, int n_shards, int64_t count_in, double eta,
                   int64_t b_cur, void* stats_inout, const float* mean_in, float* gbar_out,
                   int64_t* b_next_out, float* params, float* m, float* v,
                   const abs_adamw_hparams* hparams, int64_t step, bool fused,
                   abs_stream_t stream) {
  if (!grads || !stats_inout || !b_next_out) return ABS_ERR_NULL;
  if (count_in > 0 && !mean_in) return ABS_ERR_NULL;
  if (!fused && !gbar_out) return ABS_ERR_NULL;
  if (fused && (!params || !m || !v)) return ABS_ERR_NULL;
  if (dtype != ABS_F32 && dtype != ABS_BF16) return ABS_ERR_DTYPE;
  if (K < 1 || K > kInlineWorkers || d < 1 || b_cur < 1) return ABS_ERR_RANGE;
  if (count_in < 0 || count_in > (int64_t{1} << 40)) return ABS_ERR_RANGE;
  if (!std::isfinite(eta) || !(eta > 0.0)) return ABS_ERR_RANGE;
  if (fused) {
    const int rch = check_hparams(hparams, step);
    if (rch != ABS_OK) return rch;
  }
  const size_t esz = (dtype == ABS_F32) ? 4 : 2;
  for (int k = 0; k < K; ++k) {
    if (!grads[k]) return ABS_ERR_NULL;
    if (misaligned(grads[k], esz)) return ABS_ERR_ALIGN;
  }
  if (count_in == 0) mean_in = nullptr;  // not read
  if (misaligned(stats_inout, 16) || misaligned(b_next_out, 8) || misaligned(mean_in, 4) ||
      misaligned(gbar_out, 4))
    return ABS_ERR_ALIGN;
  if (fused && (misaligned(params, 4) || misaligned(m, 4) || misaligned(v, 4))) return ABS_ERR_ALIGN;
  Layout L;
  const int rc = make_layout(d, shard_offsets, n_shards, false, &L);
  if (rc != ABS_OK) return rc;
  const size_t ud = static_cast<size_t>(d);
  const Range outs[] = {{gbar_out, ud * 4}, {params, ud * 4}, {m, ud * 4}, {v, ud * 4},
                        {stats_inout, abs_stats_bytes(d, L.n_shards)}, {b_next_out, 8}};
  if (any_alias(grads, K, ud * esz, outs, 6)) return ABS_ERR_ALIAS;
  // the running mean may be updated in place (mean_in == gbar_out: every coordinate is read and
  // written by the same thread) but must not overlap anything else that is written
  if (mean_in)
    for (const Range& o : outs) {
      const bool in_place = o.p == gbar_out && gbar_out == mean_in;
      if (o.p && !in_place && overlaps(o.p, o.bytes, mean_in, ud * 4)) return ABS_ERR_ALIAS;
    }
  const int finalize_ctas = finalize_max_cluster();

  double* stats = static_cast<double*>(stats_inout);
  StreamParams prm;
  std::memset(&prm, 0, sizeof prm);
  for (int k = 0; k < K; ++k) prm.grads[k] = grads[k];
  std::memcpy(prm.shard_off, L.shard_off, sizeof(int64_t) * (L.n_shards + 1));
  std::memcpy(prm.chunk_prefix, L.chunk_prefix, sizeof(int32_t) * (L.n_shards + 1));
  prm.d = d;
  prm.K = K;
  prm.n_shards = L.n_shards;
  prm.n_chunks = L.n_chunks;
  prm.chunk_elems = L.chunk_elems;
  prm.gbar = gbar_out;
  prm.p = params;
  prm.m = m;
  prm.v = v;
  prm.chunk_out = stats + ABS_STATS_HEADER + static_cast<size_t>(L.n_shards) * ABS_SHARD_STRIDE;
  if (fused) prm.adam = make_adam(hparams, step);
  const double total = static_cast<double>(count_in) + static_cast<double>(K);
  AccumCarry cy;
  cy.n_prev = static_cast<double>(count_in);
  cy.inv_total = static_cast<float>(1.0 / total);
  cy.mean_in = mean_in;
  cy.shard_rec = stats + ABS_STATS_HEADER;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid(static_cast<unsigned>(L.n_chunks)), block(kThreads);
  cudaError_t e;
  // up to one group of gradients per call (16 bf16 / 8 fp32): several thread-rows in flight per
  // thread, 128 bytes of gradients or more either way (fp32: 16-byte vectors, bf16: 8-byte
  // vectors; eight rows fit for a single bf16 gradient and spill otherwise; two rows of a whole
  // group at two CTAs per SM: bf16 K=9 4.81 -> 5.77 TB/s, K=12 5.20 -> 6.22, fp32 K=5 5.15 -> 6.21).  With AdamW the state vectors are in flight as
  // well: two rows up to four gradients, one beyond.
  if (fused) {
    if (dtype == ABS_F32)
      e = K <= 4   ? launch_pdl(normtest_accumulate_kernel<F32, 2, 4, true>, grid, block, st, prm, cy)
          : K <= 8 ? launch_pdl(normtest_accumulate_kernel<F32, 1, 8, true>, grid, block, st, prm, cy)
                   : launch_pdl(normtest_accumulate_kernel<F32, 1, 1, true>, grid, block, st, prm, cy);
    else
      e = K <= 4    ? launch_pdl(normtest_accumulate_kernel<BF16H, 2, 4, true>, grid, block, st, prm, cy)
          : K <= 8  ? launch_pdl(normtest_accumulate_kernel<BF16H, 2, 8, true>, grid, block, st, prm, cy)
          : K <= 16 ? launch_pdl(normtest_accumulate_kernel<BF16H, 1, 16, true>, grid, block, st, prm, cy)
                    : launch_pdl(normtest_accumulate_kernel<BF16H, 1, 1, true>, grid, block, st, prm, cy);
  } else if (dtype == ABS_F32) {
    e = K <= 2   ? launch_pdl(normtest_accumulate_kernel<F32, 4, 2, false>, grid, block, st, prm, cy)
        : K <= 4 ? launch_pdl(normtest_accumulate_kernel<F32, 2, 4, false>, grid, block, st, prm, cy)
        : K <= 8 ? launch_pdl(normtest_accumulate_kernel<F32, 2, 8, false>, grid, block, st, prm, cy)
                 : launch_pdl(normtest_accumulate_kernel<F32, 1, 1, false>, grid, block, st, prm, cy);
  } else {
    e = K == 1   ? launch_pdl(normtest_accumulate_kernel<BF16H, 8, 1, false>, grid, block, st, prm, cy)
        : K <= 4 ? launch_pdl(normtest_accumulate_kernel<BF16H, 4, 4, false>, grid, block, st, prm, cy)
        : K <= 8 ? launch_pdl(normtest_accumulate_kernel<BF16H, 2, 8, false>, grid, block, st, prm, cy)
        : K <= 16 ? launch_pdl(normtest_accumulate_kernel<BF16H, 2, 16, false>, grid, block, st, prm, cy)
                 : launch_pdl(normtest_accumulate_kernel<BF16H, 1, 1, false>, grid, block, st, prm, cy);
  }
  if (e != cudaSuccess) return cuda_fail(e);

  FinalizeParams fp;
  std::memset(&fp, 0, sizeof fp);
  fp.chunk_in = prm.chunk_out;
  std::memcpy(fp.chunk_prefix, L.chunk_prefix, sizeof(int32_t) * (L.n_shards + 1));
  fp.n_shards = L.n_shards;
  fp.n_chunks = L.n_chunks;
  fp.stats = stats;
  fp.b_next = b_next_out;
  fp.eta = eta;
  fp.norm = total;
  fp.b_cur = b_cur;
  std::memcpy(fp.shard_first, L.shard_off, sizeof(int64_t) * L.n_shards);
  e = launch_finalize(fp, finalize_ctas, st);
  if (e != cudaSuccess) return cuda_fail(e);
  return ABS_OK;
}

// Rows per row block of the per-sample kernels: at most 512 (the row-block records then cost
// 1.6% of the matrix traffic), and, while the grid is only a few waves of 148 SMs x 3 resident
// CTAs, the count that fills whole waves (b=4096, d=16384: 13 row blocks x 32 column blocks =
// 416 of 444 CTA slots in one wave).  A function of (b, d) alone, so the shape of
// every sum is too.
int64_t persample_col_blocks(int64_t d) { return ((d + 3) / 4 + kPsThreads - 1) / kPsThreads; }

int persample_rows_per_block(int64_t b, int64_t d) {
  const int64_t wave = 148 * kPsCtasPerSM;
  const int64_t col_blocks = persample_col_blocks(d);
  const int64_t nrb_min = (b + 511) / 512;
  int64_t nrb = nrb_min;
  if (nrb_min * col_blocks < 4 * wave) {
    for (int64_t w = 1; w <= 4; ++w) {
      nrb = w * wave / col_blocks;
      if (nrb >= nrb_min) break;
    }
    if (nrb < nrb_min) nrb = nrb_min;
  }
  int64_t rpb = (b + nrb - 1) / nrb;
  // whole groups of kGroup rows (only the last row block ends in a ragged group; equal row
  // blocks that each end in a ragged group measured 1% slower)
  rpb = (rpb + kGroup - 1) / kGroup * kGroup;
  const int64_t grid_y_max = 65535;
  if ((b + rpb - 1) / rpb > grid_y_max) rpb = (b + grid_y_max - 1) / grid_y_max;
  return static_cast<int>(rpb < INT32_MAX ? rpb : INT32_MAX);
}

// The one body behind abs_persample_norm_test and its coordinate-wise form.
int run_persample(const void* G, int64_t b, int64_t d, int64_t ld, abs_dtype dtype, double eta,
                  void* stats_out, float* gbar_out, int64_t* b_next_out, bool coordwise,
                  abs_stream_t stream) {
  if (!G || !stats_out || !gbar_out || !b_next_out) return ABS_ERR_NULL;
  if (dtype != ABS_F32 && dtype != ABS_BF16) return ABS_ERR_DTYPE;
  if (b < 2 || d < 1 || ld < d) return ABS_ERR_RANGE;
  if (!std::isfinite(eta) || !(eta > 0.0)) return ABS_ERR_RANGE;
  const size_t esz = (dtype == ABS_F32) ? 4 : 2;
  if (misaligned(G, esz) || misaligned(gbar_out, 4) || misaligned(stats_out, 16) ||
      misaligned(b_next_out, 8))
    return ABS_ERR_ALIGN;
  const int64_t ncb = persample_col_blocks(d);
  const int rpb = persample_rows_per_block(b, d);
  const int64_t nrb = (b + rpb - 1) / rpb;
  if (ncb > INT32_MAX || nrb > 65535) return ABS_ERR_RANGE;
  if (overlaps(G, (static_cast<size_t>(b - 1) * ld + static_cast<size_t>(d)) * esz, gbar_out,
               static_cast<size_t>(d) * 4))
    return ABS_ERR_ALIAS;

  double* stats = static_cast<double*>(stats_out);
  PersampleParams prm;
  std::memset(&prm, 0, sizeof prm);
  prm.G = G;
  prm.b = b;
  prm.d = d;
  prm.ld = ld;
  prm.rows_per_block = rpb;
  prm.n_row_blocks = static_cast<int>(nrb);
  const int64_t nmb = (d + kPsThreads - 1) / kPsThreads;  // CTAs of the merge pass
  if (nmb > INT32_MAX) return ABS_ERR_RANGE;
  // the ticket counter sits at the same place whatever b and d are, so a buffer that has
  // served one shape (and therefore holds zero there) serves any other shape it is large enough for
  prm.tickets = reinterpret_cast<unsigned int*>(stats + ABS_STATS_HEADER + ABS_SHARD_STRIDE);
  prm.cb_rec = stats + ABS_STATS_HEADER + ABS_SHARD_STRIDE + kPsTicketDoubles;
  prm.ws_sum = prm.cb_rec + kPsRecDoubles * nmb;
  prm.ws_m2 = prm.ws_sum + nrb * d;
  prm.gbar = gbar_out;
  prm.stats = stats;
  prm.b_next = b_next_out;
  prm.eta = eta;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // rows that start on a vector boundary (16 bytes of fp32, 8 of bf16) go through the
  // asynchronous-copy ring; anything else takes element loads with the same arithmetic
  const size_t vec_bytes = 4 * esz;
  const bool ring = !misaligned(G, vec_bytes) && ((ld * esz) % vec_bytes == 0);
  const dim3 grid(static_cast<unsigned>(ncb), static_cast<unsigned>(nrb));
  const size_t ring_bytes = static_cast<size_t>(kRing) * kPsThreads * vec_bytes;
  cudaError_t e;
  if (dtype == ABS_F32)
    e = ring ? launch_pdl_smem(persample_partial_kernel<PsF32, true>, grid, dim3(kPsThreads), ring_bytes,
                               st, prm)
             : launch_pdl(persample_partial_kernel<PsF32, false>, grid, dim3(kPsThreads), st, prm);
  else
    e = ring ? launch_pdl_smem(persample_partial_kernel<PsBF16, true>, grid, dim3(kPsThreads), ring_bytes,
                               st, prm)
             : launch_pdl(persample_partial_kernel<PsBF16, false>, grid, dim3(kPsThreads), st, prm);
  if (e != cudaSuccess) return cuda_fail(e);
  const dim3 merge_grid(static_cast<unsigned>(nmb));
  e = coordwise ? launch_pdl(persample_merge_kernel<true>, merge_grid, dim3(kPsThreads), st, prm)
                : launch_pdl(persample_merge_kernel<false>, merge_grid, dim3(kPsThreads), st, prm);
  if (e != cudaSuccess) return cuda_fail(e);
  return ABS_OK;
}

}  // namespace

extern "C" {

size_t abs_stats_bytes(int64_t d, int n_shards) {
  if (d < 1 || n_shards < 1 || n_shards > ABS_MAX_SHARDS) return 0;
  const int ce = chunk_elems_for(d, true);
  const int64_t max_chunks = (d + ce - 1) / ce + n_shards;
  return sizeof(double) * (ABS_STATS_HEADER + static_cast<size_t>(n_shards) * ABS_SHARD_STRIDE +
                           static_cast<size_t>(max_chunks) * 4);
}

size_t abs_persample_stats_bytes(int64_t b, int64_t d) {
  if (b < 2 || d < 1) return 0;
  const int rpb = persample_rows_per_block(b, d);
  const size_t nrb = static_cast<size_t>((b + rpb - 1) / rpb);
  const size_t nmb = static_cast<size_t>((d + kPsThreads - 1) / kPsThreads);
  // header, one shard record, the ticket counter (two doubles' worth, at a fixed place),
  // {n2, S} per CTA of the merge pass, {sum, M2} per (row block, column)
  return sizeof(double) * (ABS_STATS_HEADER + ABS_SHARD_STRIDE + kPsTicketDoubles + kPsRecDoubles * nmb +
                           2 * nrb * static_cast<size_t>(d));
}

int abs_norm_test(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                  const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                  void* stats_out, float* gbar_out, int64_t* b_next_out, abs_stream_t stream) {
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, nullptr, nullptr, nullptr, nullptr, nullptr, 0, false,
                       stream);
}

int abs_norm_test_q(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                    const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                    void* stats_out, float* gbar_out, int64_t* b_next_out, abs_stream_t stream) {
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, nullptr, nullptr, nullptr, nullptr, nullptr, 0, false,
                       stream, false, kStatSumsQ);
}

int abs_normtest_adamw(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                       const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                       void* stats_out, float* gbar_out, int64_t* b_next_out, float* params,
                       float* m, float* v, const abs_adamw_hparams* hparams, int64_t step,
                       abs_stream_t stream) {
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, params, m, v, nullptr, hparams, step, true, stream);
}

int abs_normtest_adamw_mixed(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                             const int64_t* shard_offsets, int n_shards, double eta,
                             int64_t b_cur, void* stats_out, float* gbar_out, int64_t* b_next_out,
                             float* params, float* m, float* v, void* params_bf16_out,
                             const abs_adamw_hparams* hparams, int64_t step, abs_stream_t stream) {
  if (!params_bf16_out) return ABS_ERR_NULL;
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, params, m, v, params_bf16_out, hparams, step, true,
                       stream);
}

int abs_norm_test_coordwise(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                            const int64_t* shard_offsets, int n_shards, double eta, int64_t b_cur,
                            void* stats_out, float* gbar_out, int64_t* b_next_out,
                            abs_stream_t stream) {
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, nullptr, nullptr, nullptr, nullptr, nullptr, 0, false,
                       stream, false, kStatCoordwise);
}

int abs_normtest_adamw_coordwise(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                                 const int64_t* shard_offsets, int n_shards, double eta,
                                 int64_t b_cur, void* stats_out, float* gbar_out,
                                 int64_t* b_next_out, float* params, float* m, float* v,
                                 const abs_adamw_hparams* hparams, int64_t step,
                                 abs_stream_t stream) {
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, params, m, v, nullptr, hparams, step, true, stream,
                       false, kStatCoordwise);
}

int abs_normtest_adamw_clip_prev(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                                 const int64_t* shard_offsets, int n_shards, double eta,
                                 int64_t b_cur, void* stats_out, float* gbar_out,
                                 int64_t* b_next_out, float* params, float* m, float* v,
                                 const abs_adamw_hparams* hparams, int64_t step, double max_norm,
                                 const void* stats_prev, abs_stream_t stream) {
  const double* n2_prev = nullptr;
  if (stats_prev) {
    if (!std::isfinite(max_norm) || !(max_norm > 0.0)) return ABS_ERR_RANGE;
    if (misaligned(stats_prev, 8)) return ABS_ERR_ALIGN;
    n2_prev = static_cast<const double*>(stats_prev) + ABS_STAT_N2;
  }
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, params, m, v, nullptr, hparams, step, true, stream,
                       false, kStatSums, n2_prev, max_norm);
}

namespace {
int run_adamw(float* params, const float* gbar, float* m, float* v, int64_t d,
              const abs_adamw_hparams* hparams, int64_t step, const double* n2_dev,
              double max_norm, void* params_bf16, abs_stream_t stream) {
  if (!params || !gbar || !m || !v) return ABS_ERR_NULL;
  if (d < 1) return ABS_ERR_RANGE;
  const int rc = check_hparams(hparams, step);
  if (rc != ABS_OK) return rc;
  if (misaligned(params, 4) || misaligned(gbar, 4) || misaligned(m, 4) || misaligned(v, 4))
    return ABS_ERR_ALIGN;
  if (params_bf16 && misaligned(params_bf16, 2)) return ABS_ERR_ALIGN;
  uint16_t* p16 = static_cast<uint16_t*>(params_bf16);
  // From 2^25 coordinates on, the update runs as the fused step with one fp32 "worker" -- gbar
  // itself, whose mean over one value is that value -- and no statistics: the bulk-staged
  // kernel with its element-wise fallbacks for ragged and misaligned buffers (d = 124M: 6.86 ->
  // 6.90 TB/s, 1.24G: 6.87 -> 6.98).  Below that the plain kernel further down is faster
  // (d = 16.8M: 6.60 vs 6.50 TB/s; d = 16K: 2.3 vs 3.8 us).  Both do the same arithmetic, so the
  // results do not depend on which one ran.
  if (d >= (int64_t{1} << 25)) {
    Layout L;
    const int rcl = make_layout(d, nullptr, 1, true, &L);
    if (rcl != ABS_OK) return rcl;
    StreamParams prm;
    std::memset(&prm, 0, sizeof prm);
    prm.grads[0] = gbar;
    std::memcpy(prm.shard_off, L.shard_off, sizeof(int64_t) * 2);
    std::memcpy(prm.chunk_prefix, L.chunk_prefix, sizeof(int32_t) * 2);
    prm.d = d;
    prm.K = 1;
    prm.n_shards = 1;
    prm.n_chunks = L.n_chunks;
    prm.chunk_elems = L.chunk_elems;
    prm.inv_K = 1.0;
    prm.inv_Kf = 1.f;
    prm.neg_Kf = -1.f;
    prm.p = params;
    prm.m = m;
    prm.v = v;
    prm.p16 = p16;
    prm.clip_n2 = n2_dev;
    prm.clip_max_norm = max_norm;
    prm.adam = make_adam(hparams, step);
    const cudaError_t e1 = launch_one<F32, 1, true, true, kStatNone>(
        prm, static_cast<cudaStream_t>(stream));
    return e1 == cudaSuccess ? ABS_OK : cuda_fail(e1);
  }
  const AdamScalars a = make_adam(hparams, step);
  const bool vec = !(misaligned(params, 16) || misaligned(gbar, 16) || misaligned(m, 16) ||
                     misaligned(v, 16) || (p16 && misaligned(p16, 8)));
  // one CTA per 2048 vectors (two per thread), so CTAs retire and are replaced
  // continuously, as in the streaming kernels; a grid-stride loop covers huge d
  const int64_t work = vec ? (d + 3) / 4 : d;
  int64_t blocks = (work + 2 * kThreads - 1) / (2 * kThreads);
  const int64_t cap = int64_t{1} << 22;
  if (blocks > cap) blocks = cap;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const dim3 grid(static_cast<unsigned>(blocks)), block(kThreads);
  const cudaError_t e =
      vec ? launch_pdl(adamw_kernel<true>, grid, block, st, params, gbar, m, v, d, a, n2_dev,
                       max_norm, p16)
          : launch_pdl(adamw_kernel<false>, grid, block, st, params, gbar, m, v, d, a, n2_dev,
                       max_norm, p16);
  if (e != cudaSuccess) return cuda_fail(e);
  return ABS_OK;
}
}  // namespace

int abs_adamw_step(float* params, const float* gbar, float* m, float* v, int64_t d,
                   const abs_adamw_hparams* hparams, int64_t step, abs_stream_t stream) {
  return run_adamw(params, gbar, m, v, d, hparams, step, nullptr, 0.0, nullptr, stream);
}

int abs_adamw_step_clipped(float* params, const float* gbar, float* m, float* v, int64_t d,
                           const abs_adamw_hparams* hparams, int64_t step, double max_norm,
                           const void* stats_in, abs_stream_t stream) {
  if (!stats_in) return ABS_ERR_NULL;
  if (!std::isfinite(max_norm) || !(max_norm > 0.0)) return ABS_ERR_RANGE;
  if (misaligned(stats_in, 8)) return ABS_ERR_ALIGN;
  return run_adamw(params, gbar, m, v, d, hparams, step,
                   static_cast<const double*>(stats_in) + ABS_STAT_N2, max_norm, nullptr, stream);
}

int abs_adamw_step_mixed(float* params, const float* gbar, float* m, float* v,
                         void* params_bf16_out, int64_t d, const abs_adamw_hparams* hparams,
                         int64_t step, double max_norm, const void* stats_in,
                         abs_stream_t stream) {
  if (!params_bf16_out) return ABS_ERR_NULL;
  const double* n2_dev = nullptr;
  if (stats_in) {
    if (!std::isfinite(max_norm) || !(max_norm > 0.0)) return ABS_ERR_RANGE;
    if (misaligned(stats_in, 8)) return ABS_ERR_ALIGN;
    n2_dev = static_cast<const double*>(stats_in) + ABS_STAT_N2;
  }
  return run_adamw(params, gbar, m, v, d, hparams, step, n2_dev, stats_in ? max_norm : 0.0,
                   params_bf16_out, stream);
}

int abs_persample_norm_test(const void* G, int64_t b, int64_t d, int64_t ld, abs_dtype dtype,
                            double eta, void* stats_out, float* gbar_out, int64_t* b_next_out,
                            abs_stream_t stream) {
  return run_persample(G, b, d, ld, dtype, eta, stats_out, gbar_out, b_next_out, false, stream);
}

int abs_persample_norm_test_coordwise(const void* G, int64_t b, int64_t d, int64_t ld,
                                      abs_dtype dtype, double eta, void* stats_out,
                                      float* gbar_out, int64_t* b_next_out, abs_stream_t stream) {
  return run_persample(G, b, d, ld, dtype, eta, stats_out, gbar_out, b_next_out, true, stream);
}

int64_t abs_decide(double S, double n2, double norm, double eta, int64_t b_cur, double* T_out,
                   int* flags_out) {
  int flags = 0;
  const double T = (S / norm) / ((eta * eta) * n2);
  int64_t b_next = b_cur;
  if (!std::isfinite(S) || !std::isfinite(n2)) {
    flags |= ABS_FLAG_NONFINITE;
  } else {
    if (n2 == 0.0) flags |= ABS_FLAG_DEGENERATE;
    if (T > static_cast<double>(b_cur)) {
      flags |= ABS_FLAG_VIOLATED;
      b_next = (T >= 4611686018427387904.0) ? INT64_MAX : static_cast<int64_t>(std::ceil(T));
    }
  }
  if (T_out) *T_out = T;
  if (flags_out) *flags_out = flags;
  return b_next;
}

int64_t abs_combine_sums(const double* per_rank, int n_ranks, double norm, double eta,
                         int64_t b_cur, double* totals_out, double* T_out, int* flags_out) {
  if (!per_rank || n_ranks < 1) {
    if (T_out) *T_out = std::nan("");
    if (flags_out) *flags_out = 0;
    return -1;
  }
  double tot[3] = {0.0, 0.0, 0.0};
  for (int r = 0; r < n_ranks; ++r)  // rank order, the order in which shard records are added
    for (int j = 0; j < 3; ++j) tot[j] += per_rank[3 * r + j];
  if (totals_out)
    for (int j = 0; j < 3; ++j) totals_out[j] = tot[j];
  return abs_decide(tot[1], tot[0], norm, eta, b_cur, T_out, flags_out);
}

int64_t abs_round_batch(int64_t b_next, int64_t J, int64_t M) {
  if (b_next < 1 || J < 1 || M < 1) return -1;
  const int64_t jm = J * M;
  const int64_t micro = (b_next + jm - 1) / jm;
  return J * (M * micro);
}

int abs_selftest_bounded_wait(int polls, int64_t* out, abs_stream_t stream) {
  if (!out) return ABS_ERR_NULL;
  if (polls < 1 || polls > kBulkWaitLimit) return ABS_ERR_RANGE;
  if (misaligned(out, 8)) return ABS_ERR_ALIGN;
  const cudaError_t e = launch_pdl(bounded_wait_selftest_kernel, dim3(1), dim3(32),
                                   static_cast<cudaStream_t>(stream), polls,
                                   reinterpret_cast<long long*>(out));
  return e == cudaSuccess ? ABS_OK : cuda_fail(e);
}

const char* abs_status_string(int status) {
  switch (status) {
    case ABS_OK: return "ok";
    case ABS_ERR_NULL: return "a required pointer is NULL";
    case ABS_ERR_RANGE: return "an argument is out of range";
    case ABS_ERR_SHARDS: return "shard offsets are not a non-decreasing cover of [0, d]";
    case ABS_ERR_ALIGN: return "a buffer is not aligned to its element size";
    case ABS_ERR_DTYPE: return "unsupported dtype";
    case ABS_ERR_CUDA: return "a CUDA call failed (see abs_last_cuda_error)";
    case ABS_ERR_TOO_LARGE:
      return "the problem needs more chunk records than the built-in scratch holds "
             "(ABS_NOALLOC_MAX_CHUNKS); use abs_normtest_adamw with a caller-sized stats_out";
    case ABS_ERR_ALIAS:
      return "an output buffer overlaps a gradient buffer or another output buffer";
    default: return "unknown status";
  }
}

int abs_last_cuda_error(void) { return g_last_cuda_error; }

}  // extern "C"

extern "C" {

int abs_norm_test_accumulate(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                             const int64_t* shard_offsets, int n_shards, int64_t count_in,
                             double eta, int64_t b_cur, void* stats_inout, float* mean_inout,
                             int64_t* b_next_out, abs_stream_t stream) {
  if (!mean_inout) return ABS_ERR_NULL;
  return run_accumulate(grads, K, d, dtype, shard_offsets, n_shards, count_in, eta, b_cur,
                        stats_inout, mean_inout, mean_inout, b_next_out, nullptr, nullptr, nullptr,
                        nullptr, 0, false, stream);
}

int abs_norm_test_accumulate_adamw(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                                   const int64_t* shard_offsets, int n_shards, int64_t count_in,
                                   double eta, int64_t b_cur, void* stats_inout,
                                   const float* mean_in, float* gbar_out, int64_t* b_next_out,
                                   float* params, float* m, float* v,
                                   const abs_adamw_hparams* hparams, int64_t step,
                                   abs_stream_t stream) {
  return run_accumulate(grads, K, d, dtype, shard_offsets, n_shards, count_in, eta, b_cur,
                        stats_inout, mean_in, gbar_out, b_next_out, params, m, v, hparams, step,
                        true, stream);
}

int abs_noalloc_fits(int64_t d, const int64_t* shard_offsets, int n_shards) {
  if (d < 1) return 0;
  Layout L;
  if (make_layout(d, shard_offsets, n_shards, true, &L) != ABS_OK) return 0;
  return L.n_chunks <= ABS_NOALLOC_MAX_CHUNKS ? 1 : 0;
}

int abs_normtest_adamw_noalloc(const void* const* grads, int K, int64_t d, abs_dtype dtype,
                               const int64_t* shard_offsets, int n_shards, double eta,
                               int64_t b_cur, void* stats_out, float* gbar_out,
                               int64_t* b_next_out, float* params, float* m, float* v,
                               const abs_adamw_hparams* hparams, int64_t step,
                               abs_stream_t stream) {
  return run_norm_test(grads, K, d, dtype, shard_offsets, n_shards, eta, b_cur, stats_out,
                       gbar_out, b_next_out, params, m, v, nullptr, hparams, step, true, stream,
                       /*builtin_records=*/true);
}

}  // extern "C"
