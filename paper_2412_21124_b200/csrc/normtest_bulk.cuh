// Bulk-async (TMA 1-D) variant of the streaming norm-test kernel.
//
// Same arithmetic, same chunk records and same finalize kernel as normtest_stream_kernel;
// what changes is how the bytes move.  A full, 16-byte aligned chunk is cut into tiles of
// kBulkTile coordinates.  One elected thread issues `cp.async.bulk` copies of the tile's
// K gradient segments and (fused) p, m, v segments from global memory into a shared-memory
// stage and arms the stage's mbarrier with the byte count; all 256 threads wait on that
// mbarrier, take 4 coordinates each from shared memory, do the per-coordinate math in
// registers, write p, m, v (and gbar) back into the stage, and the elected thread sends them
// to global memory with bulk stores (the test alone, which writes only gbar, stores it straight
// from registers and keeps nothing but gradients in its stages).  kBulkStages stages keep the next tiles' loads in
// flight while a tile is computed.  Measured on the K=8 bf16 fused step this request pattern
// sustains about 2.5% more bandwidth than 128-bit loads issued per thread (the copy engine
// issues large, aligned requests and the SM spends no load/store instructions on them).
//
// Chunks that are short (end of a shard) or not 16-byte aligned take the register-direct
// path of normtest_stream.cuh inside the same kernel.  No cluster, no multicast: every
// copy is from this GPU's global memory into the issuing CTA's own shared memory.
//
// Every wait on an mbarrier is bounded.  If a wait ever runs out (it cannot unless a copy
// is lost), the CTA stops waiting, keeps its control flow uniform, drains its own copies,
// and poisons its chunk record with NaN so that the call reports ABS_FLAG_NONFINITE.
#pragma once
#include "normtest_stream.cuh"

namespace absnt {

// mbarrier polls before giving up.  A poll that fails returns after the hardware's own
// suspend time, measured at 3.95 us on a B200, so the limit is about one second: four orders
// of magnitude above any wait a landing copy needs, short enough to end a lost one soon.
constexpr int kBulkWaitLimit = 1 << 18;
constexpr int kSmemPerSM = 224 * 1024;   // budget for dynamic shared memory per SM

// bytes of one stage of `tile` coordinates
template <typename GT, int KB, bool ADAM>
__host__ __device__ constexpr int bulk_stage_bytes(int tile) {
  // fused: the K gradient segments, p, m, v and gbar; the test alone: the gradients only
  return tile * (KB * static_cast<int>(sizeof(typename GT::scalar)) + (ADAM ? 16 : 0));
}
// Shape of the staged kernel for one (dtype, K, fused) combination: coordinates per stage
// (4 per thread), stages per CTA, CTAs per SM.  tile == 0: not offered.  Measured and
// rejected: a single resident CTA with three stages (bf16 K=16: 5.83 vs 6.63 TB/s of the
// register-direct kernel) and two CTAs with two stages (bf16 K=32: 5.85 vs 6.31 TB/s).
struct BulkShape {
  int tile, stages, ctas;
};
template <typename GT, int KB, bool ADAM>
__host__ __device__ constexpr BulkShape bulk_shape() {
  // The test alone has small stages (no optimizer state), so three CTAs of three or more
  // stages fit for up to 12 bf16 / 6 fp32 workers: 24 warps per SM instead of 16 cover the
  // per-tile barrier and the wait for a tile's arrival better (bf16 K=7 6.64 -> 6.91 TB/s, K=8
  // 6.70 -> 6.88, K=9, 10 +3%; fp32 K=3 6.65 -> 6.91; K=8 bf16 on 1.24G coordinates in 8 shards
  // 6.88 -> 7.11; bf16 K=6, which used to prefer the register-direct kernel, 6.64 -> 6.95; nothing
  // lost for K = 3..5).
  // The fused kernels with stages small enough for this (bf16 K <= 4, fp32 K <= 2) lose 0.4-0.9%.
  if (!ADAM && 3 * 3 * bulk_stage_bytes<GT, KB, ADAM>(1024) <= kSmemPerSM) {
    const int fit = kSmemPerSM / (3 * bulk_stage_bytes<GT, KB, ADAM>(1024));
    return {1024, fit > 5 ? 5 : fit, 3};
  }
  if (2 * 3 * bulk_stage_bytes<GT, KB, ADAM>(1024) <= kSmemPerSM) {
    // small stages (few workers): up to five of them, so that as many bytes stay in flight
    const int fit = kSmemPerSM / (2 * bulk_stage_bytes<GT, KB, ADAM>(1024));
    return {1024, fit > 5 ? 5 : fit, 2};
  }
  if (3 * 3 * bulk_stage_bytes<GT, KB, ADAM>(512) <= kSmemPerSM) return {512, 3, 3};
  return {0, 0, 0};
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait; returns false when the limit ran out
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  for (int polls = 0; polls < kBulkWaitLimit; ++polls)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// global -> this CTA's shared memory, completion counted on `bar` (addresses and size are
// multiples of 16 bytes)
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes,
                                          uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
          "r"(smem_addr(dst_smem)),
      "l"(src), "r"(bytes), "r"(smem_addr(bar))
      : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
               "r"(smem_addr(src_smem)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_stores_read() {  // sources may be overwritten
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void bulk_wait_stores_done() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void fence_generic_to_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// 4 consecutive gradient values of worker k for this thread, from the stage
template <typename GT>
struct BulkGrad;
template <>
struct BulkGrad<BF16> {
  uint2 r;  // 4 x bf16
  __device__ __forceinline__ void load(const unsigned char* seg, int tid) {
    r = *reinterpret_cast<const uint2*>(seg + tid * 8);
  }
  __device__ __forceinline__ float elem(int j) const {
    const uint32_t w = (j >> 1) ? r.y : r.x;
    return (j & 1) ? bf16_hi(w) : bf16_lo(w);
  }
  __device__ __forceinline__ float2 pair(int jp) const {  // coordinates 2jp, 2jp+1
    const uint32_t w = jp ? r.y : r.x;
    return make_float2(bf16_lo(w), bf16_hi(w));
  }
};
template <>
struct BulkGrad<F32> {
  float4 r;
  __device__ __forceinline__ void load(const unsigned char* seg, int tid) {
    r = *reinterpret_cast<const float4*>(seg + tid * 16);
  }
  __device__ __forceinline__ float elem(int j) const {
    return j == 0 ? r.x : j == 1 ? r.y : j == 2 ? r.z : r.w;
  }
  __device__ __forceinline__ float2 pair(int jp) const {
    return jp ? make_float2(r.z, r.w) : make_float2(r.x, r.y);
  }
};

template <typename GT, int KB, bool EXACT, bool ADAM, int STAT, int TILE, int STAGES, int CTAS>
__global__ void __launch_bounds__(TILE / 4, CTAS)
    normtest_bulk_kernel(const __grid_constant__ StreamParams prm) {
  constexpr bool WITHQ = STAT == kStatSumsQ;
  constexpr bool CW = STAT == kStatCoordwise;
  constexpr int kBulkTile = TILE;
  constexpr int kBulkStages = STAGES;
  constexpr int NT = TILE / 4;  // threads
  constexpr int GB = kBulkTile * static_cast<int>(sizeof(typename GT::scalar));  // gradient segment
  constexpr int FB = kBulkTile * 4;                                              // fp32 segment
  constexpr int OFF_P = KB * GB, OFF_M = OFF_P + (ADAM ? FB : 0), OFF_V = OFF_M + (ADAM ? FB : 0);
  constexpr int OFF_GBAR = OFF_V + (ADAM ? FB : 0);
  constexpr int STAGE = OFF_GBAR + (ADAM ? FB : 0);
  static_assert(STAGE == bulk_stage_bytes<GT, KB, ADAM>(TILE), "stage layout");
  extern __shared__ __align__(128) unsigned char stages[];
  __shared__ uint64_t full[kBulkStages];
  __shared__ double red[(NT / 32) * 3];

  const int K = EXACT ? KB : prm.K;
  const int tid = threadIdx.x;
  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kBulkStages; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  uint32_t tiles_done = 0;  // tiles this CTA has consumed so far: stage and phase bookkeeping
  bool waited = false;
  bool lost = false;        // a bounded wait ran out
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
    cw.init(tid * 4);
    const bool bulk = cg.aligned && (cg.hi - cg.lo == prm.chunk_elems) &&
                      (prm.chunk_elems % kBulkTile == 0);
    if (!bulk) {
      cw.init(tid * GT::kVec);
      chunk_rows_direct<GT, KB, EXACT, ADAM, STAT, NT>(prm, K, cg, acc_n2, acc_S, acc_Q, cw, gw);
    } else {
      const int n_tiles = prm.chunk_elems / kBulkTile;
      const uint32_t tx_bytes = static_cast<uint32_t>(K * GB + (ADAM ? 3 * FB : 0));
      auto issue_loads = [&](int i) {  // elected thread only
        const uint32_t it = tiles_done + static_cast<uint32_t>(i);
        const int s = static_cast<int>(it % kBulkStages);
        unsigned char* st = stages + static_cast<size_t>(s) * STAGE;
        const int64_t e = cg.lo + static_cast<int64_t>(i) * kBulkTile;
        mbar_expect_tx(&full[s], tx_bytes);
#pragma unroll
        for (int k = 0; k < KB; ++k)
          if (EXACT || k < K)
            bulk_load(st + k * GB, reinterpret_cast<const typename GT::scalar*>(prm.grads[k]) + e,
                      GB, &full[s]);
        if (ADAM) {
          bulk_load(st + OFF_P, prm.p + e, FB, &full[s]);
          bulk_load(st + OFF_M, prm.m + e, FB, &full[s]);
          bulk_load(st + OFF_V, prm.v + e, FB, &full[s]);
        }
      };
      if (tid == 0)
        for (int j = 0; j < kBulkStages - 1 && j < n_tiles; ++j) issue_loads(j);

      for (int i = 0; i < n_tiles; ++i) {
        if (tid == 0 && i + kBulkStages - 1 < n_tiles) {
          // the stage about to be refilled was the source of the previous tile's stores
          bulk_wait_stores_read();
          issue_loads(i + kBulkStages - 1);
        }
        const uint32_t it = tiles_done + static_cast<uint32_t>(i);
        const int s = static_cast<int>(it % kBulkStages);
        if (!lost) lost = !mbar_wait_bounded(&full[s], (it / kBulkStages) & 1u);
        unsigned char* st = stages + static_cast<size_t>(s) * STAGE;

        BulkGrad<GT> raw[KB];
#pragma unroll
        for (int k = 0; k < KB; ++k)
          if (EXACT || k < K) raw[k].load(st + k * GB, tid);
        float4 pw, pm, pv;
        if (ADAM) {
          pw = *reinterpret_cast<const float4*>(st + OFF_P + tid * 16);
          pm = *reinterpret_cast<const float4*>(st + OFF_M + tid * 16);
          pv = *reinterpret_cast<const float4*>(st + OFF_V + tid * 16);
        }
        float2* w2 = reinterpret_cast<float2*>(&pw);
        float2* m2 = reinterpret_cast<float2*>(&pm);
        float2* v2 = reinterpret_cast<float2*>(&pv);
        float gb[4];
        float row_n2 = 0.f, row_S = 0.f, row_Q = 0.f;
        // two coordinates per packed instruction; the row sums take the coordinates in
        // index order, as the register-direct path does
#pragma unroll
        for (int jp = 0; jp < 2; ++jp) {
          float2 g[KB];
#pragma unroll
          for (int k = 0; k < KB; ++k)
            g[k] = (EXACT || k < K) ? raw[k].pair(jp) : make_float2(0.f, 0.f);
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
            const int li = i * kBulkTile + tid * 4 + 2 * jp;
            cw.update(dev2.x, mean.x, li);
            cw.update(dev2.y, mean.y, li + 1);
          }
          if (ADAM) adamw_pair(prm.adam, gw.omb1, gw.omb2, mean, w2[jp], m2[jp], v2[jp]);
        }
        acc_n2 += static_cast<double>(row_n2);
        acc_S += static_cast<double>(row_S);
        if (WITHQ) acc_Q += static_cast<double>(row_Q);

        if constexpr (ADAM) {
          *reinterpret_cast<float4*>(st + OFF_P + tid * 16) = pw;
          *reinterpret_cast<float4*>(st + OFF_M + tid * 16) = pm;
          *reinterpret_cast<float4*>(st + OFF_V + tid * 16) = pv;
          // the bf16 copy (mixed precision) goes straight from registers: 2 bytes per
          // coordinate do not earn a stage segment
          if (prm.p16)
            st_bf16x4(prm.p16 + cg.lo + static_cast<int64_t>(i) * kBulkTile + tid * 4, pw);
          if (prm.gbar)
            *reinterpret_cast<float4*>(st + OFF_GBAR + tid * 16) =
                make_float4(gb[0], gb[1], gb[2], gb[3]);
          fence_generic_to_async_smem();
          __syncthreads();  // tile consumed by everyone, results visible to the copy engine
          if (tid == 0) {
            const int64_t e = cg.lo + static_cast<int64_t>(i) * kBulkTile;
            bulk_store(prm.p + e, st + OFF_P, FB);
            bulk_store(prm.m + e, st + OFF_M, FB);
            bulk_store(prm.v + e, st + OFF_V, FB);
            if (prm.gbar) bulk_store(prm.gbar + e, st + OFF_GBAR, FB);
            bulk_commit();
          }
        } else {
          // the test alone writes only gbar (4 of K*s + 4 bytes per coordinate): straight from
          // registers, so that the stage holds nothing but gradients (smaller stages: more of
          // them, or a third CTA, fit) -- +0.5% at bf16 K=8 by itself
          st_stream_16(prm.gbar + cg.lo + static_cast<int64_t>(i) * kBulkTile + tid * 4,
                       make_float4(gb[0], gb[1], gb[2], gb[3]));
          __syncthreads();  // tile consumed by everyone: its stage may be refilled
        }
      }
      tiles_done += static_cast<uint32_t>(n_tiles);
      // the stages are reused by the next chunk of this CTA, and shared memory must stay
      // valid until the copy engine has read it
      if (tid == 0) bulk_wait_stores_read();
    }
    if (lost) acc_S = __longlong_as_double(0x7ff8000000000000ll);  // poison: a copy was lost
    write_chunk_record<STAT, NT>(prm, chunk, cg.lo, acc_n2, acc_S, acc_Q, cw, red);
  }
  if (tid == 0) {
    bulk_wait_stores_done();
    if (lost && tiles_done > 0) {
      // give loads that are still in flight one more bounded chance to land before the
      // shared memory is released: poll the last phase armed on every stage
#pragma unroll
      for (int s = 0; s < kBulkStages; ++s) {
        if (tiles_done <= static_cast<uint32_t>(s)) continue;
        const uint32_t last = ((tiles_done - 1 - s) / kBulkStages) * kBulkStages + s;  // last tile on s
        mbar_wait_bounded(&full[s], (last / kBulkStages) & 1u);
      }
    }
  }
}

}  // namespace absnt
