// Launch helpers and the (dtype, worker count, mode) -> kernel dispatch of the streaming
// norm-test kernels.  launch_stream<GT, ADAM, STAT> is instantiated once per combination in a
// translation unit of its own (stream_inst.cu, compiled once per combination), so that the
// ~50 kernels of each combination build in parallel; abs_api.cu only declares them.
#pragma once
#include <cstdint>
#include <mutex>
#include <type_traits>
#include <unordered_map>
#include <utility>

#include "abs_device.cuh"
#include "normtest_bulk.cuh"
#include "normtest_stream.cuh"

namespace absnt {

// Launch with the programmatic-stream-serialization attribute (see grid_dependency_wait).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st,
                       Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Raises a kernel's dynamic shared-memory limit once per (kernel, device): the attribute call
// costs about a microsecond of host time, which a launch-bound small-d loop would pay per step.
inline cudaError_t allow_dynamic_smem(const void* kernel, size_t smem) {
  static std::mutex mu;
  static std::unordered_map<const void*, uint64_t> done;  // kernel -> bit per device
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const uint64_t bit = dev < 64 ? (uint64_t{1} << dev) : 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    auto it = done.find(kernel);
    if (bit && it != done.end() && (it->second & bit)) return cudaSuccess;
  }
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  done[kernel] |= bit;
  return cudaSuccess;
}

// Launch with dynamic shared memory above the 48 KB default.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_smem(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                            cudaStream_t st, Args&&... args) {
  cudaError_t e = allow_dynamic_smem(reinterpret_cast<const void*>(kernel), smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// One (dtype, K) instantiation: the bulk-async kernel where its stages leave room for two or
// three CTAs per SM, else the register-direct kernel.
template <typename GT, int KB, bool EXACT, bool ADAM, int STAT>
cudaError_t launch_one(const StreamParams& prm, cudaStream_t st) {
  const dim3 grid(static_cast<unsigned>(prm.n_chunks));
  // Measured exceptions.  Fused: the 512-coordinate tile loses to the register-direct kernel
  // when the worker loop is predicated (EXACT false; K=12: 5.46 vs 5.80 TB/s).  Unfused test
  // (K*s + 4 bytes per coordinate, so more coordinates per second and more instructions per
  // byte): staging wins for every worker count from 3 up (by 1-9%; with three resident CTAs,
  // see bulk_shape, also for bf16 K=6 and for K=8 with the diagnostic Q or the coordinate-wise
  // maximum, which two CTAs had left to the register-direct kernel) and loses for one or two
  // workers, where the register-direct kernel is at its best (bf16 K=1 -37%, K=2 -1%; fp32 K=2
  // equal).
  constexpr BulkShape shape = bulk_shape<GT, KB, ADAM>();
  constexpr bool staged_test = EXACT && KB >= 3;
  constexpr int tile = ADAM ? ((shape.tile == 512 && !EXACT) ? 0 : shape.tile)
                            : (staged_test ? shape.tile : 0);
  if constexpr (tile > 0) {
    constexpr size_t smem =
        static_cast<size_t>(shape.stages) * bulk_stage_bytes<GT, KB, ADAM>(tile);
    return launch_pdl_smem(
        normtest_bulk_kernel<GT, KB, EXACT, ADAM, STAT, tile, shape.stages, shape.ctas>, grid,
        dim3(tile / 4), smem, st, prm);
  } else {
    return launch_pdl(normtest_stream_kernel<GT, KB, EXACT, ADAM, STAT>, grid, dim3(kThreads), st,
                      prm);
  }
}

// More than 16 workers: the split kernel, four coordinates per thread-row (bf16 gradients
// are then read with 8-byte loads).  KB bounds the worker count of the instantiation.
template <typename GT, bool EXACT, bool ADAM, int STAT, int KB = 32>
cudaError_t launch_split(const StreamParams& prm, cudaStream_t st) {
  using G4 = typename std::conditional<std::is_same<GT, BF16>::value, BF16H, GT>::type;
  return launch_pdl(normtest_split_kernel<G4, KB, EXACT, ADAM, STAT>,
                    dim3(static_cast<unsigned>(prm.n_chunks)), dim3(kThreads), st, prm);
}

// The fused kernel leaves Q out (its stats slot reads NaN): at the power cap the K extra
// multiply-adds per coordinate cost about 1% of bandwidth.  The unfused test computes it.
template <typename GT, bool ADAM, int STAT>
cudaError_t launch_stream(const StreamParams& prm, const WideTable* wide, cudaStream_t st) {
  const int K = prm.K;
  if (K > kInlineWorkers) {
    // 65..ABS_MAX_WORKERS buffers: the pointer table is a kernel parameter of its own
    using G4 = typename std::conditional<std::is_same<GT, BF16>::value, BF16H, GT>::type;
    return launch_pdl(normtest_split_wide_kernel<G4, ADAM, STAT>,
                      dim3(static_cast<unsigned>(prm.n_chunks)), dim3(kThreads), st, prm, *wide);
  }
  switch (K) {
    // every count up to 16 has an unrolled kernel of its own (one kernel for a range of counts,
    // predicating the absent workers, ran 10-25% slower: bf16 K=12 5.6 vs 6.9 TB/s, fp32 K=6
    // 5.5 vs 7.1)
    case 1: return launch_one<GT, 1, true, ADAM, STAT>(prm, st);
    case 2: return launch_one<GT, 2, true, ADAM, STAT>(prm, st);
    case 3: return launch_one<GT, 3, true, ADAM, STAT>(prm, st);
    case 4: return launch_one<GT, 4, true, ADAM, STAT>(prm, st);
    case 5: return launch_one<GT, 5, true, ADAM, STAT>(prm, st);
    case 6: return launch_one<GT, 6, true, ADAM, STAT>(prm, st);
    case 7: return launch_one<GT, 7, true, ADAM, STAT>(prm, st);
    case 8: return launch_one<GT, 8, true, ADAM, STAT>(prm, st);
    case 9: return launch_one<GT, 9, true, ADAM, STAT>(prm, st);
    case 10: return launch_one<GT, 10, true, ADAM, STAT>(prm, st);
    case 11: return launch_one<GT, 11, true, ADAM, STAT>(prm, st);
    case 12: return launch_one<GT, 12, true, ADAM, STAT>(prm, st);
    case 13: return launch_one<GT, 13, true, ADAM, STAT>(prm, st);
    case 14: return launch_one<GT, 14, true, ADAM, STAT>(prm, st);
    case 15: return launch_one<GT, 15, true, ADAM, STAT>(prm, st);
    case 16: return launch_one<GT, 16, true, ADAM, STAT>(prm, st);
    case 32: return launch_split<GT, true, ADAM, STAT>(prm, st);
    case 64:  // bf16: four unrolled groups of 16; fp32 spills in that form and takes the loop
      if constexpr (std::is_same<GT, BF16>::value) return launch_split<GT, true, ADAM, STAT, 64>(prm, st);
      else return launch_split<GT, false, ADAM, STAT, kInlineWorkers>(prm, st);
    case 17: return launch_split<GT, true, ADAM, STAT, 17>(prm, st);
    case 18: return launch_split<GT, true, ADAM, STAT, 18>(prm, st);
    case 19: return launch_split<GT, true, ADAM, STAT, 19>(prm, st);
    case 20: return launch_split<GT, true, ADAM, STAT, 20>(prm, st);
    case 21: return launch_split<GT, true, ADAM, STAT, 21>(prm, st);
    case 22: return launch_split<GT, true, ADAM, STAT, 22>(prm, st);
    case 23: return launch_split<GT, true, ADAM, STAT, 23>(prm, st);
    case 24: return launch_split<GT, true, ADAM, STAT, 24>(prm, st);
    case 25: return launch_split<GT, true, ADAM, STAT, 25>(prm, st);
    case 26: return launch_split<GT, true, ADAM, STAT, 26>(prm, st);
    case 27: return launch_split<GT, true, ADAM, STAT, 27>(prm, st);
    case 28: return launch_split<GT, true, ADAM, STAT, 28>(prm, st);
    case 29: return launch_split<GT, true, ADAM, STAT, 29>(prm, st);
    case 30: return launch_split<GT, true, ADAM, STAT, 30>(prm, st);
    case 31: return launch_split<GT, true, ADAM, STAT, 31>(prm, st);
    case 48:
      if constexpr (std::is_same<GT, BF16>::value) return launch_split<GT, true, ADAM, STAT, 48>(prm, st);
      else return launch_split<GT, false, ADAM, STAT, kInlineWorkers>(prm, st);
#define ABS_SPLIT_BF16_CASE(N)                                                              \
  case N:                                                                                   \
    if constexpr (std::is_same<GT, BF16>::value) return launch_split<GT, true, ADAM, STAT, N>(prm, st); \
    else return launch_split<GT, false, ADAM, STAT, kInlineWorkers>(prm, st);
    // the multiples of four above 32 (J workers x M accumulation steps is one in practice)
    ABS_SPLIT_BF16_CASE(36)
    ABS_SPLIT_BF16_CASE(40)
    ABS_SPLIT_BF16_CASE(44)
    ABS_SPLIT_BF16_CASE(52)
    ABS_SPLIT_BF16_CASE(56)
    ABS_SPLIT_BF16_CASE(60)
#undef ABS_SPLIT_BF16_CASE
    default:
      // 33..63 workers without a kernel of their own: run-time groups and unpredicated pieces
      // (5.6-6.1 TB/s; a kernel with compile-time groups runs at 6.4-6.7, as K = 17..32 show)
      return launch_split<GT, false, ADAM, STAT, kInlineWorkers>(prm, st);
  }
}


}  // namespace absnt
