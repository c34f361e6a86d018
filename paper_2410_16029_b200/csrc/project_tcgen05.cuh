// Projection R = P^T G (or R = G Q for a matrix projected on the right) with 256 x 256 output tiles, Sec. 1.
//
// With 128-row tiles every 256-column panel of the gradient is fetched once per 128 rows of the output.  Here one
// CTA holds two 128-row halves of the output in TMEM (2 x 256 columns, all of it) and feeds both from the same
// staged panel of B, which cuts the operand bytes per output by a third (measured: 0.99 -> 0.94 ms on r' = 512,
// K = 2048 shapes; sharing B across an SM pair as well brought nothing more).  The price is that TMEM has no
// second buffer, so the epilogue of a tile does not overlap the MMAs of the next one (the operand loads of the
// next tile do run ahead); with K in the thousands the MMAs of a tile take several times longer than its epilogue.  The host picks this kernel when
// nearly all of the work has at least 512 output rows and K >= 1536, else the 128-row kernel of gemm_tcgen05.cuh.
//
// A (K-major, bf16): Pt16 (r' x M) or G (M x N); B (N contiguous, bf16): G (M x N) or Q (N x r'); the same tensor
// maps as the 128-row kernel.  Warp roles: warp 0 TMA producer, warp 1 TMEM owner and MMA issuer, warps 2..9
// epilogue (warps 2..5 drain the upper half, 6..9 the lower; warp % 4 selects the TMEM lane quarter).  The
// epilogue transposes 32 x 32 blocks through an XOR-swizzled shared-memory block per warp and writes coalesced
// rows, with vector atomics where K is split.  Every mbarrier wait is bounded (see mbar_wait).
#pragma once

#include "gemm_tcgen05.cuh"
#include "project_gram_tcgen05.cuh"

namespace ngalore {

constexpr int kP2BN = 256;
constexpr int kP2Stages = 3;
constexpr int kP2Threads = 64 + 32 * 8;

struct P2Smem {
  static constexpr int kABytes = kTcBM * kTcBK * 2;                 // 16 KB per 128-row half
  static constexpr int kBChunkBytes = 64 * kTcBK * 2;               // 8 KB: 64 columns x 64 K rows
  static constexpr int kStageBytes = 2 * kABytes + (kP2BN / 64) * kBChunkBytes;  // 64 KB
  static constexpr int kEpiWarpBytes = 32 * 32 * 4;                 // one 32 x 32 block, swizzled
  static constexpr int kEpiOffset = kP2Stages * kStageBytes;
  static constexpr int kBarOffset = kEpiOffset + 8 * kEpiWarpBytes;
  static constexpr int kTotal = kBarOffset + 256 + 1024;            // barriers + slack for 1024-byte alignment
};
static_assert(P2Smem::kTotal <= 232448, "shared memory budget of one CTA");

__global__ void __launch_bounds__(kP2Threads, 1)
tc_project2_kernel(const CUtensorMap* __restrict__ tmaps, const TcTile* __restrict__ tiles, int n_tiles,
                   const MatDesc* __restrict__ mats, Ctrl* ctrl) {
  using L = P2Smem;
  extern __shared__ unsigned char tc_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* full_bar = bars;                    // [kP2Stages]
  uint64_t* empty_bar = bars + kP2Stages;       // [kP2Stages]
  uint64_t* tfull_bar = bars + 2 * kP2Stages;   // accumulators complete
  uint64_t* tempty_bar = tfull_bar + 1;         // accumulators drained (eight arrivals)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kP2Stages; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    mbar_init(tfull_bar, 1);
    mbar_init(tempty_bar, 8);
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
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += stride) {
        const TcTile tile = tiles[t];
        const CUtensorMap* mapA = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_A_PROJ;
        const CUtensorMap* mapB = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_B_PROJ;
        const int halves = (tile.rows - tile.m0 > kTcBM) ? 2 : 1;
        const int n_rem = tile.cols - tile.n0;
        const int n_eff = n_rem >= kP2BN ? kP2BN : ((n_rem + 15) & ~15);
        const int nchunks = (n_eff + 63) >> 6;
        const uint32_t bytes = halves * L::kABytes + nchunks * L::kBChunkBytes;
        for (int kb = 0; kb < tile.kblocks; ++kb) {
          if (!mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sA = smem + stage * L::kStageBytes;
          mbar_expect_tx(full_bar + stage, bytes);
          const int k = tile.k0 + kb * kTcBK;
          for (int h = 0; h < halves; ++h)
            tma_load_2d(sA + h * L::kABytes, mapA, k, tile.m0 + h * kTcBM, full_bar + stage);
          unsigned char* sB = sA + 2 * L::kABytes;
          for (int c = 0; c < nchunks; ++c)
            tma_load_2d(sB + c * L::kBChunkBytes, mapB, tile.n0 + c * 64, k, full_bar + stage);
          if (++stage == kP2Stages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += stride, ++local) {
        const TcTile tile = tiles[t];
        const int halves = (tile.rows - tile.m0 > kTcBM) ? 2 : 1;
        const int n_rem = tile.cols - tile.n0;
        const int n_eff = n_rem >= kP2BN ? kP2BN : ((n_rem + 15) & ~15);
        const uint32_t idesc = instr_desc(n_eff, false, false);
        if (!mbar_wait(tempty_bar, (local & 1u) ^ 1u, abort_flag)) break;
        tc_fence_after();
        for (int kb = 0; kb < tile.kblocks; ++kb) {
          if (!mbar_wait(full_bar + stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t aaddr = smem_u32(smem + stage * L::kStageBytes);
          const uint32_t baddr = aaddr + 2 * L::kABytes;
          for (int h = 0; h < halves; ++h) {
#pragma unroll
            for (int kk = 0; kk < kTcBK / 16; ++kk) {
              const uint64_t adesc = smem_desc(aaddr + h * L::kABytes + kk * 32, 16, 1024);
              const uint64_t bdesc = smem_desc(baddr + kk * 2048, L::kBChunkBytes, 1024);
              tc_mma(tmem_base + h * kP2BN, adesc, bdesc, idesc, (kb | kk) != 0 ? 1u : 0u);
            }
          }
          tc_commit(empty_bar + stage);
          if (++stage == kP2Stages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2 .. 9)
    const int quarter = warp & 3;      // TMEM lanes 32 * quarter .. + 31 belong to this warp
    const int half = (warp - 2) >> 2;  // which 128-row half of the tile this warp drains
    float* stg = reinterpret_cast<float*>(smem + L::kEpiOffset + (warp - 2) * L::kEpiWarpBytes);
    const int sub_row = lane >> 3, sub_q = lane & 7;
    int local = 0;
    for (int t = blockIdx.x; t < n_tiles; t += stride, ++local) {
      const TcTile tile = tiles[t];
      const MatDesc& d = mats[tile.mat];
      float* out = current_gradient(d, ring_cur(ctrl, d.s));
      const int halves = (tile.rows - tile.m0 > kTcBM) ? 2 : 1;
      const int n_rem = tile.cols - tile.n0;
      const int n_eff = n_rem >= kP2BN ? kP2BN : ((n_rem + 15) & ~15);
      const int row_base = tile.m0 + half * kTcBM + quarter * 32;
      if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar, local & 1u, abort_flag))) break;
      tc_fence_after();
      if (half >= halves) {
        // nothing of this warp's half exists in the tile; it only has to hand the accumulators back
        tc_fence_before();
        if (lane == 0) mbar_arrive(tempty_bar);
        continue;
      }
      for (int c0 = 0; c0 < n_eff; c0 += 32) {
        uint32_t r[32];
        tc_ld32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(half * kP2BN + c0), r);
        tc_wait_ld();
        if (c0 + 32 >= n_eff) {
          // this warp's TMEM reads of the tile are done; with all eight arrivals the next MMAs may start
          tc_fence_before();
          if (lane == 0) mbar_arrive(tempty_bar);
        }
        // row = lane; 16-byte piece j of the row goes to piece (j ^ (row & 7)): conflict-free both ways
#pragma unroll
        for (int j = 0; j < 8; ++j)
          *reinterpret_cast<float4*>(stg + lane * 32 + ((j ^ (lane & 7)) << 2)) =
              make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                          __uint_as_float(r[4 * j + 3]));
        __syncwarp();
        const int col = tile.n0 + c0 + sub_q * 4;
        if (col < tile.cols) {
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int rr = it * 4 + sub_row;
            const int row = row_base + rr;
            if (row < tile.rows) {
              const float4 acc = *reinterpret_cast<const float4*>(stg + rr * 32 + ((sub_q ^ (rr & 7)) << 2));
              float* p = out + static_cast<long long>(row) * tile.cols + col;
              if (tile.atomic) {
                atomicAdd(reinterpret_cast<float4*>(p), acc);
              } else {
                *reinterpret_cast<float4*>(p) = acc;
              }
            }
          }
        }
        __syncwarp();
      }
    }
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

// Launch-time setup of the projection kernels (call once per plan).
inline ngalore_status tc_project_init() {
  using LP = TcSmem<kProjBN, 1, 1, kProjStages, kProjEpiWarps>;
  if (cudaFuncSetAttribute(tc_gemm_kernel<kProjBN, 1, 1, kProjStages, TC_EPI_PROJECT, kProjEpiWarps, false>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, LP::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(tc_project2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P2Smem::kTotal) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  return tc_project_gram_init();
}

// R = P^T G (or G Q) for every matrix, into the buffer of the current step (ring slot `cur`, read on the device
// from Ctrl), through the tensor maps tc_bind_buffers set up.
inline ngalore_status tc_project(TcPlan& plan, const MatDesc* d_mats, Ctrl* d_ctrl, const Hyper* d_hyper,
                                 cudaStream_t stream, int64_t* launches) {
  if (plan.n_split > 0) {
    zero_split_slots_kernel<<<dim3(64, plan.n_split), 256, 0, stream>>>(d_mats, plan.d_split_mats, d_ctrl);
    *launches += 1;
  }
  if (plan.n_tiles_pg > 0) {
    // the matrices whose Gram row comes out of the projection's epilogue, then their s x s solves
    tc_project_gram_kernel<<<plan.grid_pg, kPgThreads, PgSmem::kTotal, stream>>>(
        plan.d_maps, plan.d_tiles_pg, plan.n_tiles_pg, d_mats, plan.d_pgm, plan.d_pg_part, d_ctrl);
    pg_solve_kernel<<<plan.n_pg, 256, 0, stream>>>(d_mats, plan.d_pgm, plan.d_pg_part, plan.d_pg_list, d_ctrl, d_hyper);
    *launches += 2;
    if (plan.n_tiles_proj == 0) return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
  }
  if (plan.tall_proj) {
    tc_project2_kernel<<<plan.grid_proj, kP2Threads, P2Smem::kTotal, stream>>>(plan.d_maps, plan.d_tiles_proj,
                                                                              plan.n_tiles_proj, d_mats, d_ctrl);
  } else {
    using LP = TcSmem<kProjBN, 1, 1, kProjStages, kProjEpiWarps>;
    tc_gemm_kernel<kProjBN, 1, 1, kProjStages, TC_EPI_PROJECT, kProjEpiWarps, false>
        <<<plan.grid_proj, 64 + 32 * kProjEpiWarps, LP::kTotal, stream>>>(plan.d_maps, plan.d_tiles_proj,
                                                                          plan.n_tiles_proj, d_mats, d_ctrl, nullptr);
  }
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

}  // namespace ngalore
