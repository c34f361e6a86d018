// Grouped tensor-core GEMMs of the step for sm_100a: tcgen05.mma with the accumulator in TMEM,
// operands staged in shared memory by TMA (cp.async.bulk.tensor, 128-byte swizzle), one persistent
// warp-specialised CTA per SM.
//
//   projection       R = P^T G          A = Pt16 (r' x M, K-major), B = G (M x N, N contiguous)
//                    or, for a matrix projected on the right, R = G Q:  A = G (M x N, K = N), B = Q (N x r')
//                    epilogue: store (or atomically add, when K is split) into ring slot `cur`   (Sec. 1)
//   store mode       out = A B for a table of problems (subspace refresh)
//
// The back-projection has a kernel of its own (backproject_tcgen05.cuh) built from the same wrappers.
//
// Warp roles: warp 0 issues TMA loads, warp 1 allocates TMEM and issues the MMAs, four or eight further
// warps drain the accumulator (tcgen05.ld), transpose through shared memory and write
// coalesced rows.  Two accumulator buffers let the epilogue of one tile overlap the MMAs of the next.
// Every mbarrier wait is bounded: when it runs out the CTA raises Ctrl::timeout_flag, stops issuing
// work, and still releases its TMEM.
#pragma once

#include <cuda.h>

#include <algorithm>
#include <cstring>
#include <vector>

#include "../../include/ngalore.h"
#include "common.cuh"

namespace ngalore {

constexpr int kTcBM = 128;        // rows of one accumulator tile (TMEM lanes)
constexpr int kTcBK = 64;         // K elements per pipeline stage (one 128-byte swizzle row of bf16)
constexpr unsigned long long kTcWaitLimitNs = 2000000000ull;  // a wait on an mbarrier is abandoned after 2 s

// Generic problem of the store-mode GEMM (subspace refresh): out (out_rows x out_cols, leading dimension
// ld_out, fp32) = A B with the operands' tensor maps at tmaps[map_a + part] and tmaps[map_b + part].
struct TcProblem {
  float* out;
  int out_rows, out_cols, ld_out;
  int map_a, map_b;
  int ld16 = 0;
  // if set (problems whose K is not split only): the result is written as two bf16 parts, hi = bf16(x) and
  // lo = bf16(x - hi), rows of ld16 elements, instead of as fp32 into `out`
  __nv_bfloat16* out_hi = nullptr;
  __nv_bfloat16* out_lo = nullptr;
};

struct TcTile {
  int mat;         // matrix index (projection, W update) or problem index (store mode)
  int m0, n0;      // tile origin in the output
  int k0;          // first K element
  int kblocks;     // number of 64-wide K blocks
  int atomic;      // 1: K is split, accumulate into the output with atomics
  int rows, cols;  // extent of the output the tile belongs to
};

// Tensor maps of the step GEMMs, kTcMapsPerMat consecutive entries per matrix.
enum {
  // left projection                                        right projection
  TC_MAP_A_PROJ = 0,   // Pt16: r' rows x M (K), box 64 x 128      G: M rows x N (K)
  TC_MAP_B_PROJ = 1,   // G: M (K) rows x N, box 64 x 64           P16 = Q (bf16): N (K) rows x r'
  TC_MAP_A_BACK = 2,   // P16: M rows x r' (K), box 64 x 128       u16: M rows x r' (K)
  TC_MAP_B_BACK = 3,   // u16: r' (K) rows x N, box 64 x 64        Pt16 = Q^T (fp16): r' (K) rows x N
  TC_MAP_W_LOAD = 4,   // W (fp32): M rows x N, box 32 columns x 128 rows
  TC_MAP_W_STORE = 5,  // W (fp32): box 32 x 32
  TC_MAP_H_LOAD = 6,   // history ring (fp32) as one matrix of s * lr_rows rows x lr_cols, box 32 columns x 32 rows
  kTcMapsPerMat = 7
};

// ------------------------------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: gives up after kTcWaitLimitNs of wall time (or when another warp already gave up)
// and returns false.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const uint32_t addr = smem_u32(bar);
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    if (done) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      const unsigned long long now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kTcWaitLimitNs) break;
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (64-bit): start address, leading/stride byte offsets (>>4), descriptor
// version 1 (bits 46-47), 128-byte swizzle (value 2 in bits 61-63).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  d |= 2ull << 61;
  return d;
}
// Instruction descriptor of kind::f16: fp32 accumulator, A (K-major, or MN-major when asked) and
// B (MN-major) both bf16 or both fp16, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc(int n, bool a_mn_major, bool fp16_operands) {
  const uint32_t fmt = fp16_operands ? 0u : 1u;  // operand format field: 0 = fp16, 1 = bf16
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((a_mn_major ? 1u : 0u) << 15) | (1u << 16) |
         (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(kTcBM >> 4) << 24);
}

template <int BN, int NA, int NB, int STAGES, int NEPI>
struct TcSmem {
  static constexpr int kABytes = kTcBM * kTcBK * 2;           // 16 KB
  static constexpr int kBChunkBytes = 64 * kTcBK * 2;         // one 64-column chunk: 64 K rows x 128 B
  static constexpr int kBBytes = (BN / 64) * kBChunkBytes;    // per B operand
  static constexpr int kStageBytes = NA * kABytes + NB * kBBytes;
  static constexpr int kEpiWarpBytes = 32 * 36 * 4;           // 32 rows x (32 + 4 pad) floats
  static constexpr int kBarOffset = STAGES * kStageBytes + NEPI * kEpiWarpBytes;
  static constexpr int kTotal = kBarOffset + 256 + 1024;      // barriers + slack for 1024-byte alignment
};

enum { TC_EPI_PROJECT = 0, TC_EPI_STORE = 2 };

// NA / NB: number of 16-bit parts of A / B (1, or 2 = high and low part).  With NA = NB = 2 the products
// hi*hi, hi*lo and lo*hi are accumulated (lo*lo is below fp32 resolution).  A_MN: A is stored with its
// row index contiguous (A^T row-major), staged as two 64-row chunks like B.  F16: the operands are fp16
// (otherwise bf16); TMA moves either as opaque 16-bit elements.
template <int BN, int NA, int NB, int STAGES, int EPI, int NEPI, bool A_MN, bool F16 = false>
__global__ void __launch_bounds__(64 + 32 * NEPI, 1)
tc_gemm_kernel(const CUtensorMap* __restrict__ tmaps, const TcTile* __restrict__ tiles, int n_tiles,
               const MatDesc* __restrict__ mats, Ctrl* ctrl, const TcProblem* __restrict__ probs) {
  using L = TcSmem<BN, NA, NB, STAGES, NEPI>;
  extern __shared__ unsigned char tc_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* full_bar = bars;                   // [STAGES]
  uint64_t* empty_bar = bars + STAGES;         // [STAGES]
  uint64_t* tfull_bar = bars + 2 * STAGES;     // [2]
  uint64_t* tempty_bar = bars + 2 * STAGES + 2;  // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar + b, 1); mbar_init(tempty_bar + b, 4); }
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

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
        const TcTile tile = tiles[t];
        const CUtensorMap *mapA, *mapB0;
        int out_cols;
        if (EPI == TC_EPI_STORE) {
          const TcProblem pr = probs[tile.mat];
          mapA = tmaps + pr.map_a;
          mapB0 = tmaps + pr.map_b;
          out_cols = pr.out_cols;
        } else {
          mapA = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_A_PROJ;
          mapB0 = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_B_PROJ;
          out_cols = tile.cols;
        }
        const int n_rem = out_cols - tile.n0;
        const int n_eff = n_rem >= BN ? BN : ((n_rem + 15) & ~15);
        const int nchunks = (n_eff + 63) >> 6;
        const uint32_t bytes = NA * L::kABytes + NB * nchunks * L::kBChunkBytes;
        for (int kb = 0; kb < tile.kblocks; ++kb) {
          if (!mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sA = smem + stage * L::kStageBytes;
          mbar_expect_tx(full_bar + stage, bytes);
          const int k = tile.k0 + kb * kTcBK;
#pragma unroll
          for (int na = 0; na < NA; ++na) {
            if (A_MN) {
              tma_load_2d(sA + na * L::kABytes, mapA + na, tile.m0, k, full_bar + stage);
              tma_load_2d(sA + na * L::kABytes + L::kBChunkBytes, mapA + na, tile.m0 + 64, k, full_bar + stage);
            } else {
              tma_load_2d(sA + na * L::kABytes, mapA + na, k, tile.m0, full_bar + stage);
            }
          }
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            unsigned char* sB = sA + NA * L::kABytes + nb * L::kBBytes;
            for (int c = 0; c < nchunks; ++c)
              tma_load_2d(sB + c * L::kBChunkBytes, mapB0 + nb, tile.n0 + c * 64, k, full_bar + stage);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
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
      for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++local) {
        const TcTile tile = tiles[t];
        const int out_cols = (EPI == TC_EPI_STORE) ? probs[tile.mat].out_cols : tile.cols;
        const int n_rem = out_cols - tile.n0;
        const int n_eff = n_rem >= BN ? BN : ((n_rem + 15) & ~15);
        const uint32_t idesc = instr_desc(n_eff, A_MN, F16);
        const int buf = local & 1;
        const uint32_t tphase = (local >> 1) & 1u;
        if (!mbar_wait(tempty_bar + buf, tphase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * BN;
        for (int kb = 0; kb < tile.kblocks; ++kb) {
          if (!mbar_wait(full_bar + stage, phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t aaddr0 = smem_u32(smem + stage * L::kStageBytes);
          bool first = (kb == 0);
#pragma unroll
          for (int na = 0; na < NA; ++na) {
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
              if (na == 1 && nb == 1) continue;  // lo * lo is dropped
              const uint32_t aaddr = aaddr0 + na * L::kABytes;
              const uint32_t baddr = aaddr0 + NA * L::kABytes + nb * L::kBBytes;
#pragma unroll
              for (int kk = 0; kk < kTcBK / 16; ++kk) {
                const uint64_t adesc = A_MN ? smem_desc(aaddr + kk * 2048, L::kBChunkBytes, 1024)
                                            : smem_desc(aaddr + kk * 32, 16, 1024);
                const uint64_t bdesc = smem_desc(baddr + kk * 2048, L::kBChunkBytes, 1024);
                tc_mma(tmem_d, adesc, bdesc, idesc, first ? 0u : 1u);
                first = false;
              }
            }
          }
          tc_commit(empty_bar + stage);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(tfull_bar + buf);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2 .. 2 + NEPI - 1)
    // With 8 epilogue warps there are two groups of four; group g drains accumulator buffer g, i.e. the
    // tiles with (local & 1) == g.
    const int quarter = warp & 3;  // TMEM lanes 32 * quarter .. + 31 belong to this warp
    constexpr int kGroups = NEPI / 4;
    const int group = (warp - 2) >> 2;
    float* stg = reinterpret_cast<float*>(smem + STAGES * L::kStageBytes + (warp - 2) * L::kEpiWarpBytes);
    int local = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++local) {
      if (kGroups == 2 && (local & 1) != group) continue;
      const TcTile tile = tiles[t];
      float* out;
      __nv_bfloat16 *out_hi = nullptr, *out_lo = nullptr;
      int rows_total, out_cols, ld_out, ld16 = 0;
      if (EPI == TC_EPI_STORE) {
        const TcProblem pr = probs[tile.mat];
        out = pr.out;
        rows_total = pr.out_rows;
        out_cols = pr.out_cols;
        ld_out = pr.ld_out;
        out_hi = pr.out_hi;
        out_lo = pr.out_lo;
        ld16 = pr.ld16;
      } else {
        const MatDesc& d = mats[tile.mat];
        out_cols = tile.cols;
        ld_out = tile.cols;
        out = current_gradient(d, ring_cur(ctrl, d.s));
        rows_total = tile.rows;
      }
      const int n_rem = out_cols - tile.n0;
      const int n_eff = n_rem >= BN ? BN : ((n_rem + 15) & ~15);
      const int buf = local & 1;
      const uint32_t tphase = (local >> 1) & 1u;
      const int row_base = tile.m0 + quarter * 32;
      const int sub_row = lane >> 3, sub_col = (lane & 7) * 4;
      if (!mbar_wait(tfull_bar + buf, tphase, abort_flag)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < BN; c0 += 32) {
        if (c0 < n_eff) {
          uint32_t r[32];
          tc_ld32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(buf * BN + c0), r);
          tc_wait_ld();
          if (c0 + 32 >= n_eff) {
            // all TMEM reads of this tile are done: hand the buffer back before the global traffic
            tc_fence_before();
            if (lane == 0) mbar_arrive(tempty_bar + buf);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j)
            *reinterpret_cast<float4*>(stg + lane * 36 + j * 4) =
                make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                            __uint_as_float(r[4 * j + 3]));
          __syncwarp();
          const int col = tile.n0 + c0 + sub_col;
          if (col < out_cols) {
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              const int rr = it * 4 + sub_row;
              const int row = row_base + rr;
              if (row < rows_total) {
                const float4 acc = *reinterpret_cast<const float4*>(stg + rr * 36 + sub_col);
                float* p = out + static_cast<long long>(row) * ld_out + col;
                if (EPI == TC_EPI_STORE && out_hi != nullptr) {
                  const __nv_bfloat162 h01 = __floats2bfloat162_rn(acc.x, acc.y), h23 = __floats2bfloat162_rn(acc.z, acc.w);
                  const __nv_bfloat162 l01 = __floats2bfloat162_rn(acc.x - __low2float(h01), acc.y - __high2float(h01));
                  const __nv_bfloat162 l23 = __floats2bfloat162_rn(acc.z - __low2float(h23), acc.w - __high2float(h23));
                  uint2 hv, lv;
                  hv.x = *reinterpret_cast<const uint32_t*>(&h01); hv.y = *reinterpret_cast<const uint32_t*>(&h23);
                  lv.x = *reinterpret_cast<const uint32_t*>(&l01); lv.y = *reinterpret_cast<const uint32_t*>(&l23);
                  const long long o = static_cast<long long>(row) * ld16 + col;
                  *reinterpret_cast<uint2*>(out_hi + o) = hv;
                  *reinterpret_cast<uint2*>(out_lo + o) = lv;
                } else if (tile.atomic) {
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

// Zero the ring slot the projection is about to accumulate into, for the matrices whose K is split.
__global__ void zero_split_slots_kernel(const MatDesc* mats, const int* split_mats, const Ctrl* ctrl) {
  const MatDesc& d = mats[split_mats[blockIdx.y]];
  float4* p = reinterpret_cast<float4*>(current_gradient(d, ring_cur(ctrl, d.s)));
  const long long n4 = d.rn / 4;
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n4;
       i += static_cast<long long>(gridDim.x) * blockDim.x)
    p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

// ------------------------------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kProjBN = 256, kProjStages = 4, kProjEpiWarps = 4;
constexpr int kTcBackBN = 256;  // tile width of the back-projection kernel

// Projection with the Gram row in its epilogue (project_gram_tcgen05.cuh): tile width, the longest history that
// takes part, partial rows per tile (one per epilogue warp).
constexpr int kPgBN = 256;
constexpr int kPgSMax = 16;
constexpr int kPgWarpRows = 8;

// Per matrix: where its partial rows start in the partial buffer (in doubles; -1: the matrix does not take part)
// and its tile grid.  Partial row of (tile, epilogue warp e): part_off + (tile * 8 + e) * kPgSMax.
struct PgMat {
  long long part_off;
  int ntiles;
  int tiles_n;   // tiles per 128-row band (columns / 256, rounded up)
};

struct TcPlan {
  size_t device_bytes = 0;
  EncodeTiledFn encode = nullptr;
  int n_mats = 0;
  std::vector<CUtensorMap> h_maps;  // kTcMapsPerMat per matrix (TC_MAP_*)
  std::vector<int> rowsN;           // per matrix: M, N for re-encoding the maps of G and W
  std::vector<int> colsN;
  std::vector<int> right;           // per matrix: projected on the right
  bool tall_proj = false;           // projection tiles are 256 rows high (tc_project2_kernel)
  bool long_k_back = false;         // back-projection with three operand stages and a short W ring
  // Binding sets: the tensor maps of one particular array of G and W pointers, encoded once, kept in pinned host
  // memory and uploaded once.  A training loop that cycles through a few gradient buffers (or always passes the
  // same ones) pays for encoding and upload only the first time it shows a set; afterwards a step does no host
  // work beyond comparing the pointers.  All sets are allocated with the plan; the least recently used one is
  // overwritten when a new array of pointers arrives and every set is taken.
  struct Binding {
    std::vector<const void*> G, W;
    uint64_t hash = 0;
    bool valid = false;
    int64_t last_use = 0;
    cudaEvent_t uploaded = nullptr;  // recorded after the upload from h_pinned: the pinned copy may be rewritten after it
    CUtensorMap* d_maps = nullptr;
    CUtensorMap* h_pinned = nullptr;
  };
  std::vector<Binding> bindings;
  int64_t bind_clock = 0;
  int64_t bind_uploads = 0;         // how many times a set had to be encoded and uploaded
  CUtensorMap* d_maps_all = nullptr;
  CUtensorMap* h_pinned_all = nullptr;
  CUtensorMap* d_maps = nullptr;    // the set of the current call (one of bindings[*].d_maps)
  // Behind the tensor maps every set also carries the raw pointers (n gradient pointers, then n weight pointers) for
  // the kernels that read G and W with plain loads (small-rank path).
  size_t ptr_offset = 0;            // bytes from the start of a set to its pointers
  size_t set_bytes = 0;
  const uint16_t* const* d_Gptr = nullptr;   // of the current call
  float* const* d_Wptr = nullptr;
  TcTile* d_tiles_proj = nullptr;
  TcTile* d_tiles_back = nullptr;
  std::vector<int> back_tile0;     // first back-projection tile of every matrix, plus the total (n + 1 entries)
  int n_tiles_proj = 0, n_tiles_back = 0;
  int grid_proj = 0, grid_back = 0;
  int* d_split_mats = nullptr;
  int n_split = 0;
  // projection with the Gram row in its epilogue: the matrices that take part, their tiles and partial rows
  std::vector<int> gram_fused;     // per matrix: 1 when its Gram row comes from the projection's epilogue
  TcTile* d_tiles_pg = nullptr;
  int n_tiles_pg = 0, grid_pg = 0;
  PgMat* d_pgm = nullptr;
  double* d_pg_part = nullptr;
  int* d_pg_list = nullptr;
  int n_pg = 0;
};

// 16-bit elements unless fp32 is asked for (TMA moves fp16 and bf16 alike).
inline bool tc_encode_2d(EncodeTiledFn fn, CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer,
                         uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer, bool fp32 = false) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline void tc_plan_destroy(TcPlan& plan) {
  for (TcPlan::Binding& b : plan.bindings)
    if (b.uploaded) cudaEventDestroy(b.uploaded);
  plan.bindings.clear();
  if (plan.d_maps_all) cudaFree(plan.d_maps_all);
  if (plan.h_pinned_all) cudaFreeHost(plan.h_pinned_all);
  plan.d_maps_all = nullptr; plan.h_pinned_all = nullptr;
  if (plan.d_tiles_proj) cudaFree(plan.d_tiles_proj);
  if (plan.d_tiles_back) cudaFree(plan.d_tiles_back);
  if (plan.d_split_mats) cudaFree(plan.d_split_mats);
  if (plan.d_tiles_pg) cudaFree(plan.d_tiles_pg);
  if (plan.d_pgm) cudaFree(plan.d_pgm);
  if (plan.d_pg_part) cudaFree(plan.d_pg_part);
  if (plan.d_pg_list) cudaFree(plan.d_pg_list);
  plan.d_maps = nullptr; plan.d_tiles_proj = nullptr; plan.d_tiles_back = nullptr; plan.d_split_mats = nullptr;
  plan.d_tiles_pg = nullptr; plan.d_pgm = nullptr; plan.d_pg_part = nullptr; plan.d_pg_list = nullptr;
}

inline ngalore_status tc_plan_create(TcPlan& plan, const std::vector<MatDesc>& mats, const MatDesc* /*d_mats*/, int s,
                                     int sm_count, bool allow_gram_fusion) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr)
    return NGALORE_ERR_CUDA;
  plan.encode = reinterpret_cast<EncodeTiledFn>(fn);
  const int n = static_cast<int>(mats.size());
  plan.n_mats = n;
  plan.h_maps.resize(static_cast<size_t>(n) * kTcMapsPerMat);
  std::memset(plan.h_maps.data(), 0, sizeof(CUtensorMap) * plan.h_maps.size());
  for (int i = 0; i < n; ++i) {
    const MatDesc& d = mats[i];
    CUtensorMap* mp = &plan.h_maps[static_cast<size_t>(i) * kTcMapsPerMat];
    bool ok = true;
    if (!d.right) {
      // A_proj: Pt16, r' rows x M (K) columns, row stride ldpt
      ok &= tc_encode_2d(plan.encode, mp + TC_MAP_A_PROJ, d.Pt16, d.M, d.rp, static_cast<uint64_t>(d.ldpt) * 2, kTcBK, kTcBM);
      // A_back: P16, M rows x r' (K) columns, row stride ldp
      ok &= tc_encode_2d(plan.encode, mp + TC_MAP_A_BACK, d.P16, d.rp, d.M, static_cast<uint64_t>(d.ldp) * 2, kTcBK, kTcBM);
      // B_back: u16, r' (K) rows x N columns
      ok &= tc_encode_2d(plan.encode, mp + TC_MAP_B_BACK, d.u16, d.N, d.rp, static_cast<uint64_t>(d.N) * 2, 64, kTcBK);
    } else {
      // B_proj: Q as bf16 (P16), N (K) rows x ldp columns (those beyond r' are zero), row stride ldp
      ok &= tc_encode_2d(plan.encode, mp + TC_MAP_B_PROJ, d.P16, d.ldp, d.N, static_cast<uint64_t>(d.ldp) * 2, 64, kTcBK);
      // A_back: u16, M rows x lr_cols (K) columns (those beyond r' are zero)
      ok &= tc_encode_2d(plan.encode, mp + TC_MAP_A_BACK, d.u16, d.lr_cols, d.M, static_cast<uint64_t>(d.lr_cols) * 2, kTcBK, kTcBM);
      // B_back: Q^T as fp16 (Pt16), r' (K) rows x N columns, row stride ldpt
      ok &= tc_encode_2d(plan.encode, mp + TC_MAP_B_BACK, d.Pt16, d.N, d.rp, static_cast<uint64_t>(d.ldpt) * 2, 64, kTcBK);
    }
    if (!ok) return NGALORE_ERR_CUDA;
  }

  // ---- projection tiles: output lr_rows x lr_cols (r' x N with K = M, or M x r' with K = N when the matrix is
  // projected on the right); split K so that no tile dominates the schedule
  // Tile height: 256 rows (two 128-row halves sharing every staged panel of B, project_tcgen05.cuh) when nearly
  // all of the work sits in matrices with more than 128 output rows, else 128 rows.
  // Measured: on r = 512 shapes (K = 2048) the tall tiles bring 0.99 -> 0.94 ms, on r = 256 shapes (K = 768 or 1024,
  // one tile covers all output rows) they cost 8 %, because the epilogue no longer overlaps the next tile's MMAs.
  // The back-projection picks its shared-memory split by the length of K = r' (backproject_tcgen05.cuh).
  {
    long long work_all = 0, work_tall = 0, work_long_k = 0;
    for (int i = 0; i < n; ++i) {
      const long long w = static_cast<long long>(mats[i].M) * mats[i].N;
      work_all += w;
      if (mats[i].lr_rows >= 4 * kTcBM && (mats[i].right ? mats[i].N : mats[i].M) >= 1536) work_tall += w;
      if (mats[i].rp > 5 * kTcBK) work_long_k += w;
    }
    plan.tall_proj = work_tall * 10 >= work_all * 9;
    plan.long_k_back = work_long_k * 10 >= work_all * 9;
  }
  const int proj_bm = plan.tall_proj ? 2 * kTcBM : kTcBM;
  std::vector<TcTile> proj, back;
  long long total_kb = 0;
  for (int i = 0; i < n; ++i) {
    const MatDesc& d = mats[i];
    const long long tiles_i = static_cast<long long>((d.lr_rows + kTcBM - 1) / kTcBM) * ((d.lr_cols + kProjBN - 1) / kProjBN);
    total_kb += tiles_i * (((d.right ? d.N : d.M) + kTcBK - 1) / kTcBK);
  }
  const long long per_cta = (total_kb + sm_count - 1) / sm_count;
  long long target_kb = per_cta / 4;
  if (target_kb < 16) target_kb = 16;
  std::vector<int> split_mats;
  // Matrices whose Gram row is formed in the projection's epilogue (project_gram_tcgen05.cuh): the workload class
  // of the tall projection tiles (long K, rank 512: there the history read is long enough to hide the MMAs),
  // left projection, K short enough to stay unsplit, fp32 history of at most kPgSMax slots, rows and columns
  // multiples of 32.
  plan.gram_fused.assign(n, 0);
  std::vector<TcTile> pg;
  std::vector<PgMat> pgm(n, PgMat{-1, 0, 0});
  std::vector<int> pg_list;
  long long pg_rows = 0;
  const bool fuse_class = allow_gram_fusion && plan.tall_proj && s >= 1 && s <= kPgSMax;
  for (int i = 0; i < n; ++i) {
    const MatDesc& d = mats[i];
    const int kb_total = ((d.right ? d.N : d.M) + kTcBK - 1) / kTcBK;
    int splits = static_cast<int>((kb_total + target_kb - 1) / target_kb);
    if (splits < 1) splits = 1;
    const int kb_per = (kb_total + splits - 1) / splits;
    splits = (kb_total + kb_per - 1) / kb_per;
    // (a K of up to 128 blocks stays in one piece for it even where the schedule would rather split it)
    if (fuse_class && kb_total <= 128 && !d.right && d.H16 == nullptr && d.s == s && d.lr_rows % 32 == 0 && d.lr_cols % 32 == 0) {
      plan.gram_fused[i] = 1;
      pg_list.push_back(i);
      const int tiles_m = (d.lr_rows + kTcBM - 1) / kTcBM, tiles_n = (d.lr_cols + kPgBN - 1) / kPgBN;
      pgm[i] = PgMat{pg_rows * kPgSMax, tiles_m * tiles_n, tiles_n};
      pg_rows += static_cast<long long>(tiles_m) * tiles_n * kPgWarpRows;
      for (int n0 = 0; n0 < d.lr_cols; n0 += kPgBN)
        for (int m0 = 0; m0 < d.lr_rows; m0 += kTcBM)
          pg.push_back(TcTile{i, m0, n0, 0, kb_total, 0, d.lr_rows, d.lr_cols});
      continue;
    }
    if (splits > 1) split_mats.push_back(i);
    for (int n0 = 0; n0 < d.lr_cols; n0 += kProjBN)
      for (int sp = 0; sp < splits; ++sp)
        for (int m0 = 0; m0 < d.lr_rows; m0 += proj_bm) {
          const int kb0 = sp * kb_per;
          const int kbn = std::min(kb_per, kb_total - kb0);
          proj.push_back(TcTile{i, m0, n0, kb0 * kTcBK, kbn, splits > 1 ? 1 : 0, d.lr_rows, d.lr_cols});
        }
  }
  std::stable_sort(proj.begin(), proj.end(), [](const TcTile& a, const TcTile& b) { return a.kblocks > b.kblocks; });
  std::stable_sort(pg.begin(), pg.end(), [](const TcTile& a, const TcTile& b) { return a.kblocks > b.kblocks; });
  plan.back_tile0.assign(n + 1, 0);
  for (int i = 0; i < n; ++i) {
    const MatDesc& d = mats[i];
    plan.back_tile0[i] = static_cast<int>(back.size());
    const int kbn = (d.rp + kTcBK - 1) / kTcBK;
    for (int m0 = 0; m0 < d.M; m0 += kTcBM)
      for (int n0 = 0; n0 < d.N; n0 += kTcBackBN) back.push_back(TcTile{i, m0, n0, 0, kbn, 0, d.M, d.N});
  }
  plan.back_tile0[n] = static_cast<int>(back.size());
  plan.n_tiles_proj = static_cast<int>(proj.size());
  plan.n_tiles_back = static_cast<int>(back.size());
  plan.grid_proj = std::min(plan.n_tiles_proj, sm_count);
  plan.grid_back = std::min(plan.n_tiles_back, sm_count);
  plan.n_split = static_cast<int>(split_mats.size());
  plan.n_tiles_pg = static_cast<int>(pg.size());
  plan.grid_pg = std::min(plan.n_tiles_pg, sm_count);
  plan.n_pg = static_cast<int>(pg_list.size());
  for (int i : pg_list) {
    // the whole ring of the matrix as one tall fp32 matrix: slot j starts at row j * lr_rows
    const MatDesc& d = mats[i];
    if (!tc_encode_2d(plan.encode, &plan.h_maps[static_cast<size_t>(i) * kTcMapsPerMat + TC_MAP_H_LOAD], d.H, d.lr_cols,
                      static_cast<uint64_t>(s) * d.lr_rows, static_cast<uint64_t>(d.lr_cols) * 4, 32, 32, true))
      return NGALORE_ERR_CUDA;
  }
  if (plan.n_pg > 0) {
    if (cudaMalloc(&plan.d_tiles_pg, sizeof(TcTile) * pg.size()) != cudaSuccess) { plan.d_tiles_pg = nullptr; return NGALORE_ERR_ALLOC; }
    if (cudaMalloc(&plan.d_pgm, sizeof(PgMat) * n) != cudaSuccess) { plan.d_pgm = nullptr; return NGALORE_ERR_ALLOC; }
    if (cudaMalloc(&plan.d_pg_part, sizeof(double) * pg_rows * kPgSMax) != cudaSuccess) { plan.d_pg_part = nullptr; return NGALORE_ERR_ALLOC; }
    if (cudaMalloc(&plan.d_pg_list, sizeof(int) * pg_list.size()) != cudaSuccess) { plan.d_pg_list = nullptr; return NGALORE_ERR_ALLOC; }
    if (cudaMemcpy(plan.d_tiles_pg, pg.data(), sizeof(TcTile) * pg.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(plan.d_pgm, pgm.data(), sizeof(PgMat) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(plan.d_pg_list, pg_list.data(), sizeof(int) * pg_list.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(plan.d_pg_part, 0, sizeof(double) * pg_rows * kPgSMax) != cudaSuccess)
      return NGALORE_ERR_CUDA;
    plan.device_bytes += sizeof(TcTile) * pg.size() + sizeof(PgMat) * n + sizeof(double) * pg_rows * kPgSMax + sizeof(int) * pg_list.size();
  }

  // binding sets: as many as fit in 64 MB, between 2 and 32
  plan.ptr_offset = (sizeof(CUtensorMap) * plan.h_maps.size() + 255) / 256 * 256;
  plan.set_bytes = (plan.ptr_offset + sizeof(void*) * 2 * n + 255) / 256 * 256;
  const size_t set_bytes = plan.set_bytes;
  int n_sets = static_cast<int>((64u << 20) / set_bytes);
  n_sets = n_sets < 2 ? 2 : (n_sets > 32 ? 32 : n_sets);
  const size_t maps_bytes = set_bytes * n_sets;
  if (cudaMalloc(&plan.d_maps_all, maps_bytes) != cudaSuccess) { plan.d_maps_all = nullptr; return NGALORE_ERR_ALLOC; }
  if (cudaMallocHost(&plan.h_pinned_all, maps_bytes) != cudaSuccess) { plan.h_pinned_all = nullptr; return NGALORE_ERR_ALLOC; }
  plan.bindings.resize(n_sets);
  for (int b = 0; b < n_sets; ++b) {
    plan.bindings[b].d_maps = reinterpret_cast<CUtensorMap*>(reinterpret_cast<char*>(plan.d_maps_all) + b * set_bytes);
    plan.bindings[b].h_pinned = reinterpret_cast<CUtensorMap*>(reinterpret_cast<char*>(plan.h_pinned_all) + b * set_bytes);
    if (cudaEventCreateWithFlags(&plan.bindings[b].uploaded, cudaEventDisableTiming) != cudaSuccess) {
      plan.bindings[b].uploaded = nullptr;
      return NGALORE_ERR_CUDA;
    }
  }
  plan.d_maps = plan.bindings[0].d_maps;
  if (cudaMalloc(&plan.d_tiles_proj, sizeof(TcTile) * proj.size()) != cudaSuccess) { plan.d_tiles_proj = nullptr; return NGALORE_ERR_ALLOC; }
  if (cudaMalloc(&plan.d_tiles_back, sizeof(TcTile) * back.size()) != cudaSuccess) { plan.d_tiles_back = nullptr; return NGALORE_ERR_ALLOC; }
  if (cudaMalloc(&plan.d_split_mats, sizeof(int) * (split_mats.size() + 1)) != cudaSuccess) { plan.d_split_mats = nullptr; return NGALORE_ERR_ALLOC; }
  plan.device_bytes += maps_bytes + sizeof(TcTile) * (proj.size() + back.size()) + sizeof(int) * (split_mats.size() + 1);
  if (cudaMemcpy(plan.d_tiles_proj, proj.data(), sizeof(TcTile) * proj.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_tiles_back, back.data(), sizeof(TcTile) * back.size(), cudaMemcpyHostToDevice) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  if (!split_mats.empty() &&
      cudaMemcpy(plan.d_split_mats, split_mats.data(), sizeof(int) * split_mats.size(), cudaMemcpyHostToDevice) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  plan.rowsN.resize(n); plan.colsN.resize(n); plan.right.resize(n);
  for (int i = 0; i < n; ++i) { plan.rowsN[i] = mats[i].M; plan.colsN[i] = mats[i].N; plan.right[i] = mats[i].right; }

  return NGALORE_OK;
}

// Point the tensor maps of the step at this call's gradients and weights (host arrays of device pointers,
// 16-byte aligned, row-major M x N).  An array of pointers that was seen before (and whose binding set has not
// been overwritten since) costs a comparison of the pointers; a new one is encoded into its set's pinned host
// copy and uploaded from there, asynchronously on `stream`.
inline ngalore_status tc_bind_buffers(TcPlan& plan, const uint16_t* const* G, float* const* W, cudaStream_t stream) {
  const int n = plan.n_mats;
  uint64_t hash = 1469598103934665603ull;
  for (int i = 0; i < n; ++i) {
    hash = (hash ^ reinterpret_cast<uintptr_t>(G[i])) * 1099511628211ull;
    hash = (hash ^ reinterpret_cast<uintptr_t>(W[i])) * 1099511628211ull;
  }
  plan.bind_clock += 1;
  TcPlan::Binding* victim = nullptr;  // a free set if there is one, else the least recently used
  for (TcPlan::Binding& b : plan.bindings) {
    if (b.valid && b.hash == hash && std::equal(b.G.begin(), b.G.end(), reinterpret_cast<const void* const*>(G)) &&
        std::equal(b.W.begin(), b.W.end(), reinterpret_cast<const void* const*>(W))) {
      b.last_use = plan.bind_clock;
      plan.d_maps = b.d_maps;
      plan.d_Gptr = reinterpret_cast<const uint16_t* const*>(reinterpret_cast<char*>(b.d_maps) + plan.ptr_offset);
      plan.d_Wptr = reinterpret_cast<float* const*>(reinterpret_cast<char*>(b.d_maps) + plan.ptr_offset) + n;
      return NGALORE_OK;
    }
    if (victim == nullptr || (victim->valid && (!b.valid || b.last_use < victim->last_use))) victim = &b;
  }
  TcPlan::Binding& b = *victim;
  // the previous upload from this pinned copy must have been read before it is rewritten
  if (b.valid && cudaEventSynchronize(b.uploaded) != cudaSuccess) return NGALORE_ERR_CUDA;
  b.valid = false;
  std::memcpy(b.h_pinned, plan.h_maps.data(), sizeof(CUtensorMap) * plan.h_maps.size());
  for (int i = 0; i < n; ++i) {
    CUtensorMap* mp = b.h_pinned + static_cast<size_t>(i) * kTcMapsPerMat;
    // G is the B operand of a left projection (K = M rows) and the A operand of a right one (K = N columns)
    const bool enc = plan.right[i]
                         ? tc_encode_2d(plan.encode, mp + TC_MAP_A_PROJ, G[i], plan.colsN[i], plan.rowsN[i],
                                        static_cast<uint64_t>(plan.colsN[i]) * 2, kTcBK, kTcBM)
                         : tc_encode_2d(plan.encode, mp + TC_MAP_B_PROJ, G[i], plan.colsN[i], plan.rowsN[i],
                                        static_cast<uint64_t>(plan.colsN[i]) * 2, 64, kTcBK);
    if (!enc) return NGALORE_ERR_CUDA;
    const uint64_t row_bytes = static_cast<uint64_t>(plan.colsN[i]) * 4;
    if (!tc_encode_2d(plan.encode, mp + TC_MAP_W_LOAD, W[i], plan.colsN[i], plan.rowsN[i], row_bytes, 32, kTcBM, true) ||
        !tc_encode_2d(plan.encode, mp + TC_MAP_W_STORE, W[i], plan.colsN[i], plan.rowsN[i], row_bytes, 32, 32, true))
      return NGALORE_ERR_CUDA;
  }
  {
    const void** hp = reinterpret_cast<const void**>(reinterpret_cast<char*>(b.h_pinned) + plan.ptr_offset);
    for (int i = 0; i < n; ++i) { hp[i] = G[i]; hp[n + i] = W[i]; }
  }
  if (cudaMemcpyAsync(b.d_maps, b.h_pinned, plan.set_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaEventRecord(b.uploaded, stream) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  b.G.assign(reinterpret_cast<const void* const*>(G), reinterpret_cast<const void* const*>(G) + n);
  b.W.assign(reinterpret_cast<const void* const*>(W), reinterpret_cast<const void* const*>(W) + n);
  b.hash = hash;
  b.valid = true;
  b.last_use = plan.bind_clock;
  plan.bind_uploads += 1;
  plan.d_maps = b.d_maps;
  plan.d_Gptr = reinterpret_cast<const uint16_t* const*>(reinterpret_cast<char*>(b.d_maps) + plan.ptr_offset);
  plan.d_Wptr = reinterpret_cast<float* const*>(reinterpret_cast<char*>(b.d_maps) + plan.ptr_offset) + n;
  return NGALORE_OK;
}

}  // namespace ngalore
