// Back-projection with the weight update fused in (Sec. 2.2):  W <- (1 - lr wd) W - lr P u  for every matrix.
//
// One persistent warp-specialised CTA per SM walks 128 x 256 tiles of W.  A = P16 (M x r', fp16, K-major),
// B = u16 (r' x N, fp16), fp32 accumulator in TMEM (two buffers of 256 columns).  W never passes through
// registers as global traffic: a producer warp streams the tile into shared memory with TMA, 32 columns
// (one 16 KB slot of a short ring) at a time, while the MMAs of the tile run; the epilogue warps update each slot
// in place, row per lane, against the accumulator they read with tcgen05.ld, and one lane per warp sends
// its 32 x 32 box back with a TMA store.  The 128-byte swizzle of the W boxes makes the row-per-lane float4
// accesses free of bank conflicts, so no transposition is needed between the TMEM layout and shared memory.
// The wide tile is what keeps the operand traffic from L2 (A once per 256 columns) below the W traffic.
//
// Warp roles: warp 0 TMA producer of the operands' K blocks, warp 1 TMEM owner and MMA issuer, warps 2..9
// epilogue (warp quarter q = warp % 4 owns rows 32 q .. 32 q + 31 of the tile, the two warps of a quarter
// take the even and the odd 32-column chunks), warp 10 TMA producer of the W slots.  Every mbarrier wait is
// bounded (see mbar_wait).
#pragma once

#include "gemm_tcgen05.cuh"

namespace ngalore {

constexpr int kBpBN = kTcBackBN;        // tile columns
// Two shapes of the shared-memory budget (STAGES operand stages of 48 KB, SLOTS W slots of 128 rows x 32 columns):
//   3 stages + 5 slots where K = r' is long (six K blocks or more): measured on the 1.1B shapes (r' = 512), with two
//     stages 8 / 7 / 6 / 5 slots ran 2.12 / 2.07 / 1.97 / 1.93 ms and the memory a short ring frees for a third
//     stage brings 1.67-1.75 ms (3 stages + 4 slots 2.13 ms, + 3 slots 2.46 ms): a W producer that runs a whole
//     tile ahead takes bandwidth from the operand loads the MMAs are waiting for;
//   2 stages + 8 slots where K is short and the kernel is all W traffic (r' = 8 on the same shapes: 1.48 ms
//     against 1.58 ms with the short ring; r' = 256: 0.525 against 0.545 ms).
// At least four slots are needed: an epilogue warp releases a slot one chunk late (see below), so each of the two
// chunk parities must fit two slots.
constexpr int kBpWProducerWarp = 10;    // warps 0, 1: operand producer and MMA issuer; 2..9: epilogue; 10: W producer
constexpr int kBpThreads = 32 * 11;

template <int STAGES, int SLOTS>
struct BpSmem {
  static_assert(SLOTS >= 4, "the deferred slot release needs two slots per chunk parity");
  static_assert((2 * STAGES + 4 + 2 * SLOTS) * 8 + 8 <= 256, "barrier block");
  static constexpr int kABytes = kTcBM * kTcBK * 2;                 // 16 KB
  static constexpr int kBChunkBytes = 64 * kTcBK * 2;               // 8 KB: 64 columns x 64 K rows
  static constexpr int kStageBytes = kABytes + (kBpBN / 64) * kBChunkBytes;  // 48 KB
  static constexpr int kWBoxBytes = 32 * 32 * 4;                    // 4 KB: 32 rows x 128 B
  static constexpr int kWSlotBytes = 4 * kWBoxBytes;                // 128 rows x 32 columns
  static constexpr int kWOffset = STAGES * kStageBytes;
  static constexpr int kBarOffset = kWOffset + SLOTS * kWSlotBytes;
  static constexpr int kTotal = kBarOffset + 256 + 1024;            // barriers + slack for 1024-byte alignment
};
static_assert(BpSmem<3, 5>::kTotal <= 232448 && BpSmem<2, 8>::kTotal <= 232448, "shared memory budget of one CTA");

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, int x, int y, const void* src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(src))
               : "memory");
}

// 32-column chunks of W a tile covers.
__device__ __forceinline__ int bp_wchunks(const TcTile& tile) {
  const int n_rem = tile.cols - tile.n0;
  return n_rem >= kBpBN ? kBpBN / 32 : (n_rem + 31) >> 5;
}

template <int kBpStages, int kBpSlots>
__global__ void __launch_bounds__(kBpThreads, 1)
tc_backproject_kernel(const CUtensorMap* __restrict__ tmaps, const TcTile* __restrict__ tiles, int n_tiles,
                      const MatDesc* __restrict__ mats, Ctrl* ctrl, const Hyper* __restrict__ hyper) {
  using L = BpSmem<kBpStages, kBpSlots>;
  extern __shared__ unsigned char tc_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* full_bar = bars;                        // [kBpStages] operands landed
  uint64_t* empty_bar = bars + kBpStages;           // [kBpStages] operands consumed
  uint64_t* tfull_bar = bars + 2 * kBpStages;       // [2] accumulator complete
  uint64_t* tempty_bar = bars + 2 * kBpStages + 2;  // [2] accumulator drained
  uint64_t* wfull_bar = bars + 2 * kBpStages + 4;   // [kBpSlots] W slot landed
  uint64_t* wempty_bar = wfull_bar + kBpSlots;      // [kBpSlots] W slot sent back (its shared memory is free)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(wempty_bar + kBpSlots);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kBpStages; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar + b, 1); mbar_init(tempty_bar + b, 8); }
    for (int s = 0; s < kBpSlots; ++s) { mbar_init(wfull_bar + s, 1); mbar_init(wempty_bar + s, 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u)
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
    // ------------------------------------------------------------------ TMA producer of the W slots
    // The slots are used in the order (tile, chunk); slot and barrier phase follow from the running count.
    if (lane == 0 && static_cast<int>(blockIdx.x) < n_tiles) {
      int slot = 0;
      uint32_t phase = 0;
      TcTile tile = tiles[blockIdx.x];
      for (int t = blockIdx.x; t < n_tiles; t += stride) {
        const int tn = t + stride;
        const TcTile next = tiles[tn < n_tiles ? tn : t];
        const int wchunks = bp_wchunks(tile);
        const CUtensorMap* mapW = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_W_LOAD;
        bool ok = true;
        for (int c = 0; c < wchunks; ++c) {
          if (!mbar_wait(wempty_bar + slot, phase ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(wfull_bar + slot, L::kWSlotBytes);
          tma_load_2d(smem + L::kWOffset + slot * L::kWSlotBytes, mapW, tile.n0 + c * 32, tile.m0, wfull_bar + slot);
          if (++slot == kBpSlots) { slot = 0; phase ^= 1u; }
        }
        if (!ok) break;
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
    const int parity = (warp - 2) >> 2;  // this warp takes the chunks with (c & 1) == parity
    const float lr = hyper->lr, decay = 1.f - hyper->lr * hyper->wd;
    int slot = 0;                        // ring position of the tile's chunk 0, advanced over all chunks
    uint32_t phase = 0;
    int pending_slot = -1;               // slot whose store was issued last and is not yet released
    if (static_cast<int>(blockIdx.x) < n_tiles) {
      TcTile tile = tiles[blockIdx.x];
      int bad = __ldcg(mats[tile.mat].step_bad);
      int local = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += stride, ++local) {
        const int tn = t + stride;
        const TcTile next = tiles[tn < n_tiles ? tn : t];
        const int bad_next = __ldcg(mats[next.mat].step_bad);
        const int buf = local & 1;
        const uint32_t tphase = (local >> 1) & 1u;
        const int wchunks = bp_wchunks(tile);
        const int row0 = tile.m0 + quarter * 32;
        const bool store = !bad && row0 < tile.rows;
        const CUtensorMap* mapW = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_W_STORE;
        // every lane polls; the warp goes on only if all of them saw the barrier complete
        if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar + buf, tphase, abort_flag))) break;
        tc_fence_after();
        const int last_own = ((wchunks - 1 - parity) & ~1) + parity;  // this warp's last chunk (< parity: none)
        if (last_own < parity) {
          tc_fence_before();
          if (lane == 0) mbar_arrive(tempty_bar + buf);
        }
        for (int c = 0; c < wchunks; ++c) {
          if ((c & 1) == parity) {
            if (!__all_sync(0xffffffffu, mbar_wait(wfull_bar + slot, phase, abort_flag))) { ok = false; break; }
            uint32_t r[32];
            tc_ld32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(buf * kBpBN + c * 32), r);
            tc_wait_ld();
            if (c == last_own) {
              // this warp's TMEM reads of the tile are done; with all eight arrivals the next MMAs may start
              tc_fence_before();
              if (lane == 0) mbar_arrive(tempty_bar + buf);
            }
            // this lane's row of the 32 x 32 box: 16-byte piece j sits at piece (j ^ (row & 7)) of the 128-byte row
            unsigned char* box = smem + L::kWOffset + slot * L::kWSlotBytes + quarter * L::kWBoxBytes;
            unsigned char* rowp = box + lane * 128;
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
            // hand the updated rows to the async proxy, then one lane stores the box; the slot is released
            // once the store has read it, which inside a tile is checked one chunk later so that the warp
            // does not idle
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
              if (store) {
                tma_store_2d(mapW, tile.n0 + c * 32, row0, box);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                if (pending_slot >= 0) {
                  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                  mbar_arrive(wempty_bar + pending_slot);
                }
                pending_slot = slot;
              } else {
                mbar_arrive(wempty_bar + slot);
              }
            }
            __syncwarp();
          }
          if (++slot == kBpSlots) { slot = 0; phase ^= 1u; }
        }
        // No release stays pending across tiles: the W producer may need the slot before this warp's next
        // chunk comes up (a narrow tile can leave a warp without a chunk of its own).
        if (lane == 0 && pending_slot >= 0) {
          asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          mbar_arrive(wempty_bar + pending_slot);
          pending_slot = -1;
        }
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
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// Launch-time setup of the kernel above (call once per plan).
inline ngalore_status tc_backproject_init() {
  if (cudaFuncSetAttribute(tc_backproject_kernel<3, 5>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           BpSmem<3, 5>::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(tc_backproject_kernel<2, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           BpSmem<2, 8>::kTotal) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  return NGALORE_OK;
}

// W <- (1 - lr wd) W - lr P u for the matrices [mat0, mat1), through the tensor maps tc_bind_buffers set up.
inline ngalore_status tc_backproject_range(TcPlan& plan, int mat0, int mat1, const MatDesc* d_mats, Ctrl* d_ctrl,
                                           const Hyper* d_hyper, cudaStream_t stream, int64_t* launches) {
  const int t0 = plan.back_tile0[mat0], t1 = plan.back_tile0[mat1];
  if (t1 <= t0) return NGALORE_OK;
  const int grid = (t1 - t0) < plan.grid_back ? (t1 - t0) : plan.grid_back;
  if (plan.long_k_back)
    tc_backproject_kernel<3, 5><<<grid, kBpThreads, BpSmem<3, 5>::kTotal, stream>>>(plan.d_maps, plan.d_tiles_back + t0,
                                                                                   t1 - t0, d_mats, d_ctrl, d_hyper);
  else
    tc_backproject_kernel<2, 8><<<grid, kBpThreads, BpSmem<2, 8>::kTotal, stream>>>(plan.d_maps, plan.d_tiles_back + t0,
                                                                                   t1 - t0, d_mats, d_ctrl, d_hyper);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

// W <- (1 - lr wd) W - lr P u for every matrix.
inline ngalore_status tc_backproject(TcPlan& plan, const MatDesc* d_mats, Ctrl* d_ctrl, const Hyper* d_hyper,
                                     cudaStream_t stream, int64_t* launches) {
  return tc_backproject_range(plan, 0, plan.n_mats, d_mats, d_ctrl, d_hyper, stream, launches);
}

}  // namespace ngalore
