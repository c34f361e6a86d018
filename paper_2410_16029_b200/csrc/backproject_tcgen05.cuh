// Back-projection with the weight update fused in (Sec. 2.2):  W <- (1 - lr wd) W - lr P u  for every matrix.
//
// One persistent warp-specialised CTA per SM walks 128 x 128 tiles of W.  A = P16 (M x r', fp16, K-major),
// B = u16 (r' x N, fp16), fp32 accumulator in TMEM (two buffers).  W never passes through registers as
// global traffic: the producer warp brings the W tile into shared memory with TMA while the MMAs of the
// tile (and the epilogue of the previous one) run, the epilogue warps update it in place, row per lane,
// against the accumulator they read with tcgen05.ld, and one lane per warp sends the 32 x 32 boxes back
// with TMA stores.  The 128-byte swizzle of the W boxes makes the row-per-lane float4 accesses free of
// bank conflicts, so no transposition is needed between the TMEM layout and shared memory.
//
// Warp roles: warp 0 TMA producer of the operands' K blocks, warp 1 TMEM owner and MMA issuer, warps 2..9
// epilogue in two groups of four (group g owns accumulator buffer g and W buffer g, i.e. every second tile
// of the CTA), warp 10 TMA producer of the W tiles, so that a wait for a W buffer never holds up the
// operand pipeline.  Every mbarrier wait is bounded (see mbar_wait).
#pragma once

#include "gemm_tcgen05.cuh"

namespace ngalore {

constexpr int kBpBN = 128;      // tile columns
constexpr int kBpStages = 3;    // operand pipeline depth
constexpr int kBpWProducerWarp = 10;  // warps 0, 1: operand producer and MMA issuer; 2..9: epilogue; 10: W producer
constexpr int kBpThreads = 32 * 11;

struct BpSmem {
  static constexpr int kABytes = kTcBM * kTcBK * 2;                 // 16 KB
  static constexpr int kBChunkBytes = 64 * kTcBK * 2;               // 8 KB: 64 columns x 64 K rows
  static constexpr int kStageBytes = kABytes + (kBpBN / 64) * kBChunkBytes;  // 32 KB
  static constexpr int kWBoxBytes = 32 * 32 * 4;                    // 4 KB: 32 rows x 128 B
  static constexpr int kWChunkBytes = 4 * kWBoxBytes;               // 128 rows x 32 columns
  static constexpr int kWBufBytes = (kBpBN / 32) * kWChunkBytes;    // 64 KB
  static constexpr int kWOffset = kBpStages * kStageBytes;
  static constexpr int kBarOffset = kWOffset + 2 * kWBufBytes;
  static constexpr int kTotal = kBarOffset + 256 + 1024;            // barriers + slack for 1024-byte alignment
};
static_assert(BpSmem::kTotal <= 232448, "shared memory budget of one CTA");

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, const void* src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(src))
               : "memory");
}

__global__ void __launch_bounds__(kBpThreads, 1)
tc_backproject_kernel(const CUtensorMap* __restrict__ tmaps, const TcTile* __restrict__ tiles, int n_tiles,
                      const MatDesc* __restrict__ mats, Ctrl* ctrl, const Hyper* __restrict__ hyper) {
  using L = BpSmem;
  extern __shared__ unsigned char tc_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* full_bar = bars;                        // [kBpStages] operands landed
  uint64_t* empty_bar = bars + kBpStages;           // [kBpStages] operands consumed
  uint64_t* tfull_bar = bars + 2 * kBpStages;       // [2] accumulator complete
  uint64_t* tempty_bar = bars + 2 * kBpStages + 2;  // [2] accumulator drained
  uint64_t* wfull_bar = bars + 2 * kBpStages + 4;   // [2] W tile landed
  uint64_t* wempty_bar = bars + 2 * kBpStages + 6;  // [2] W tile sent back (its shared memory is free)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kBpStages + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kBpStages; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar + b, 1);
      mbar_init(tempty_bar + b, 4);
      mbar_init(wfull_bar + b, 1);
      mbar_init(wempty_bar + b, 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int stride = gridDim.x;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer of the operands
    if (lane == 0 && static_cast<int>(blockIdx.x) < n_tiles) {
      int stage = 0;
      uint32_t phase = 0;
      TcTile tile = tiles[blockIdx.x];
      for (int t = blockIdx.x; t < n_tiles; t += stride) {
        const int tn = t + stride;
        const TcTile next = tiles[tn < n_tiles ? tn : t];  // fetched early: its latency hides behind this tile
        const CUtensorMap* maps = tmaps + tile.mat * kTcMapsPerMat;
        const int n_rem = tile.cols - tile.n0;
        const int n_eff = n_rem >= kBpBN ? kBpBN : ((n_rem + 15) & ~15);
        const int nchunks = (n_eff + 63) >> 6;
        const uint32_t bytes = L::kABytes + nchunks * L::kBChunkBytes;
        bool ok = true;
        for (int kb = 0; kb < tile.kblocks; ++kb) {
          if (!mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sA = smem + stage * L::kStageBytes;
          mbar_expect_tx(full_bar + stage, bytes);
          const int k = kb * kTcBK;
          tma_load_2d(sA, maps + TC_MAP_A_BACK, k, tile.m0, full_bar + stage);
          for (int c = 0; c < nchunks; ++c)
            tma_load_2d(sA + L::kABytes + c * L::kBChunkBytes, maps + TC_MAP_B_BACK, tile.n0 + c * 64, k, full_bar + stage);
          if (++stage == kBpStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tile = next;
      }
    }
  } else if (warp == kBpWProducerWarp) {
    // ------------------------------------------------------------------ TMA producer of the W tiles
    if (lane == 0 && static_cast<int>(blockIdx.x) < n_tiles) {
      int local = 0;
      TcTile tile = tiles[blockIdx.x];
      for (int t = blockIdx.x; t < n_tiles; t += stride, ++local) {
        const int tn = t + stride;
        const TcTile next = tiles[tn < n_tiles ? tn : t];
        const int buf = local & 1;
        const uint32_t wphase = (local >> 1) & 1u;
        const int n_rem = tile.cols - tile.n0;
        const int wchunks = n_rem >= kBpBN ? kBpBN / 32 : (n_rem + 31) >> 5;
        if (!mbar_wait(wempty_bar + buf, wphase ^ 1u, abort_flag)) break;
        mbar_expect_tx(wfull_bar + buf, static_cast<uint32_t>(wchunks) * L::kWChunkBytes);
        unsigned char* sW = smem + L::kWOffset + buf * L::kWBufBytes;
        const CUtensorMap* mapW = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_W_LOAD;
        for (int c = 0; c < wchunks; ++c)
          tma_load_2d(sW + c * L::kWChunkBytes, mapW, tile.n0 + c * 32, tile.m0, wfull_bar + buf);
        tile = next;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && static_cast<int>(blockIdx.x) < n_tiles) {
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      TcTile tile = tiles[blockIdx.x];
      for (int t = blockIdx.x; t < n_tiles; t += stride, ++local) {
        const int tn = t + stride;
        const TcTile next = tiles[tn < n_tiles ? tn : t];
        const int n_rem = tile.cols - tile.n0;
        const int n_eff = n_rem >= kBpBN ? kBpBN : ((n_rem + 15) & ~15);
        const uint32_t idesc = instr_desc(n_eff, false, true);
        const int buf = local & 1;
        const uint32_t tphase = (local >> 1) & 1u;
        if (!mbar_wait(tempty_bar + buf, tphase ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * kBpBN;
        bool ok = true;
        for (int kb = 0; kb < tile.kblocks; ++kb) {
          if (!mbar_wait(full_bar + stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t aaddr = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t baddr = aaddr + L::kABytes;
#pragma unroll
          for (int kk = 0; kk < kTcBK / 16; ++kk) {
            const uint64_t adesc = smem_desc(aaddr + kk * 32, 16, 1024);
            const uint64_t bdesc = smem_desc(baddr + kk * 2048, L::kBChunkBytes, 1024);
            tc_mma(tmem_d, adesc, bdesc, idesc, (kb | kk) != 0 ? 1u : 0u);
          }
          tc_commit(empty_bar + stage);
          if (++stage == kBpStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar + buf);
        tile = next;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2 .. 9)
    const int quarter = warp & 3;        // TMEM lanes 32 * quarter .. + 31 belong to this warp
    const int group = (warp - 2) >> 2;   // accumulator / W buffer this warp's group owns
    const float lr = hyper->lr, decay = 1.f - hyper->lr * hyper->wd;
    unsigned char* sW = smem + L::kWOffset + group * L::kWBufBytes + quarter * L::kWBoxBytes;
    const int first = blockIdx.x + group * stride;
    if (first < n_tiles) {
      TcTile tile = tiles[first];
      int bad = __ldcg(mats[tile.mat].step_bad);
      int it = 0;
      for (int t = first; t < n_tiles; t += 2 * stride, ++it) {
        const int tn = t + 2 * stride;
        const TcTile next = tiles[tn < n_tiles ? tn : t];
        const int bad_next = __ldcg(mats[next.mat].step_bad);
        const uint32_t ph = it & 1u;
        const int n_rem = tile.cols - tile.n0;
        const int wchunks = n_rem >= kBpBN ? kBpBN / 32 : (n_rem + 31) >> 5;
        // every lane polls; the warp goes on only if all of them saw both barriers complete
        bool ready = mbar_wait(wfull_bar + group, ph, abort_flag);
        ready = ready && mbar_wait(tfull_bar + group, ph, abort_flag);
        if (!__all_sync(0xffffffffu, ready)) break;
        tc_fence_after();
        for (int c = 0; c < wchunks; ++c) {
          uint32_t r[32];
          tc_ld32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(group * kBpBN + c * 32), r);
          tc_wait_ld();
          if (c == wchunks - 1) {
            // all TMEM reads of this tile are done: the MMAs of the group's next tile may start
            tc_fence_before();
            if (lane == 0) mbar_arrive(tempty_bar + group);
          }
          // this lane's row of the 32 x 32 box: 16-byte piece j sits at piece (j ^ (row & 7)) of the 128-byte row
          unsigned char* rowp = sW + c * L::kWChunkBytes + lane * 128;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            float4* p = reinterpret_cast<float4*>(rowp + ((j ^ (lane & 7)) << 4));
            float4 w = *p;
            w.x = decay * w.x - lr * __uint_as_float(r[4 * j]);
            w.y = decay * w.y - lr * __uint_as_float(r[4 * j + 1]);
            w.z = decay * w.z - lr * __uint_as_float(r[4 * j + 2]);
            w.w = decay * w.w - lr * __uint_as_float(r[4 * j + 3]);
            *p = w;
          }
        }
        // hand the updated rows to the async proxy, then one lane stores the warp's boxes
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          const int row0 = tile.m0 + quarter * 32;
          if (!bad && row0 < tile.rows) {
            const CUtensorMap* mapW = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_W_STORE;
            for (int c = 0; c < wchunks; ++c) tma_store_2d(mapW, tile.n0 + c * 32, row0, sW + c * L::kWChunkBytes);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          }
          mbar_arrive(wempty_bar + group);
        }
        __syncwarp();
        tile = next;
        bad = bad_next;
      }
    }
    // the stores must have reached memory before the CTA retires
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a wait ran out: give bulk copies that may still be in flight time to land before the CTA retires
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    if (threadIdx.x == 0) atomicExch(&ctrl->timeout_flag, 1);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
  }
}

// Launch-time setup of the kernel above (call once per plan).
inline ngalore_status tc_backproject_init() {
  return cudaFuncSetAttribute(tc_backproject_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BpSmem::kTotal) == cudaSuccess
             ? NGALORE_OK
             : NGALORE_ERR_CUDA;
}

// W <- (1 - lr wd) W - lr P u for every matrix, through the tensor maps tc_bind_buffers set up.
inline ngalore_status tc_backproject(TcPlan& plan, const MatDesc* d_mats, Ctrl* d_ctrl, const Hyper* d_hyper,
                                     cudaStream_t stream, int64_t* launches) {
  tc_backproject_kernel<<<plan.grid_back, kBpThreads, BpSmem::kTotal, stream>>>(
      plan.d_maps, plan.d_tiles_back, plan.n_tiles_back, d_mats, d_ctrl, d_hyper);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

}  // namespace ngalore
