// Projection R = P^T G with the new row of the history's Gram matrix formed in its epilogue (Sec. 1; Sec. 2.4:
// y = G^T g, the inner products of the current low-rank gradient with the stacked past ones).  Option
// gram_fusion; off by default because it measured slower than the separate kernels as built.
//
// The Gram row needs one read of the whole history ring, which is HBM traffic with no arithmetic to speak of,
// and the projection is tensor-core time with little traffic.  Run one after the other neither hides the other;
// here every epilogue warp streams the older ring slots of the rows it is draining through a small ring of its
// own in shared memory (TMA boxes of 32 rows x 32 columns, 128-byte swizzle: the row-per-lane float4 reads are
// conflict-free), a few boxes ahead and across tile boundaries, while the MMAs of the next tile run into the
// second accumulator buffer.  Each epilogue thread holds its row of a 32-column chunk of R from tcgen05.ld,
// writes it to the ring slot of the current step and multiplies it into the same piece of every older slot.
// Products and the per-thread sums over a tile are fp32, everything across threads is fp64, as in the stream
// kernel's Gram pass.  Every epilogue warp writes its partial row per tile (no synchronisation between warps);
// pg_solve_kernel, launched behind this kernel, adds the partial rows of a matrix in a fixed order, solves the
// s x s system and publishes the weights for the combination pass.
//
// Only matrices whose R comes out of a single CTA per tile take part (left projection, K of at most 128 blocks so
// that it stays unsplit, row and column counts multiples of 32, 1 <= s <= 16, fp32 history); the others keep the
// plain projection and the Gram tiles of the stream kernel.
//
// Warp roles: warp 0 TMA producer of the operands, warp 1 TMEM owner and MMA issuer, warps 2..9 epilogue
// (quarter = warp % 4 owns 32 rows; the two warps of a quarter take the even and the odd 32-column chunks).
// Every mbarrier wait is bounded (see mbar_wait).
#pragma once

#include "backproject_tcgen05.cuh"
#include "kernels_stream.cuh"

namespace ngalore {

constexpr int kPgThreads = 32 * 10;

// Inner product of a thread's 32 accumulator columns with 32 values of the same row of another matrix, in one
// fixed order of operations (see the epilogue).
__device__ __forceinline__ float pg_dot32(const uint32_t (&r)[32], const float4 (&h)[8]) {
  float t = 0.f;
#pragma unroll
  for (int q = 0; q < 8; ++q)
    t += __uint_as_float(r[4 * q]) * h[q].x + __uint_as_float(r[4 * q + 1]) * h[q].y +
         __uint_as_float(r[4 * q + 2]) * h[q].z + __uint_as_float(r[4 * q + 3]) * h[q].w;
  return t;
}

// Three operand stages of 48 KB and two history boxes of 4 KB in flight per epilogue warp.  Measured on the 1.1B
// shapes (kernel + solves + the embeddings' plain projection): 2 stages with 4 boxes per warp 2.93 ms, 3 stages
// with 2 boxes 2.78 ms: under a saturated memory system the operand loads of the MMAs are what the kernel waits
// for.  An earlier arrangement with a producer warp and 16 KB boxes shared by four warps (128 rows) ran 2.96 ms.
constexpr int kPgStages = 3;      // operand stages of 48 KB
constexpr int kPgBoxes = 2;       // boxes in flight per epilogue warp
struct PgSmem {
  static constexpr int kABytes = kTcBM * kTcBK * 2;
  static constexpr int kBChunkBytes = 64 * kTcBK * 2;
  static constexpr int kStageBytes = kABytes + (kPgBN / 64) * kBChunkBytes;   // 48 KB
  static constexpr int kBoxBytes = 32 * 32 * 4;                               // 4 KB
  static constexpr int kRingOffset = kPgStages * kStageBytes;
  static constexpr int kBarOffset = kRingOffset + 8 * kPgBoxes * kBoxBytes;
  static constexpr int kBarBytes = 512;
  static constexpr int kTotal = kBarOffset + kBarBytes + 1024;
};
static_assert((2 * kPgStages + 4 + 8 * kPgBoxes) * 8 + 8 <= PgSmem::kBarBytes, "barrier block");
static_assert(PgSmem::kTotal <= 232448, "shared memory budget of one CTA");

// Walks the boxes of one epilogue warp in the order it uses them: tile (this CTA's), older slot, own chunk
// (slot-major, so that DRAM sees 1 KB of a row within a few boxes: measured 2.78 ms against 3.03 ms chunk-major).
struct PgBoxIter {
  int t, j, c, wchunks;
  int n0, m0, rows, mat;
  bool valid;
};
__device__ __forceinline__ int pg_next_slot(int j, int cur, int count) {
  ++j;
  if (j == cur) ++j;
  return j < count ? j : -1;
}
__device__ __forceinline__ void pg_iter_load_tile(PgBoxIter& it, const TcTile* tiles) {
  const TcTile tile = tiles[it.t];
  const int n_rem = tile.cols - tile.n0;
  it.wchunks = (n_rem >= kPgBN ? kPgBN : n_rem) >> 5;
  it.n0 = tile.n0; it.m0 = tile.m0; it.rows = tile.rows; it.mat = tile.mat;
}
// First box at or after tile it.t (tiles that have no chunk of this warp's parity are skipped).
__device__ __forceinline__ void pg_iter_seek(PgBoxIter& it, const TcTile* tiles, int n_tiles, int stride, int parity,
                                             int cur, int count) {
  it.valid = false;
  if (count < 2) return;
  while (it.t < n_tiles) {
    pg_iter_load_tile(it, tiles);
    if (parity < it.wchunks) {
      it.j = pg_next_slot(-1, cur, count);
      it.c = parity;
      it.valid = true;
      return;
    }
    it.t += stride;
  }
}
__device__ __forceinline__ void pg_iter_advance(PgBoxIter& it, const TcTile* tiles, int n_tiles, int stride, int parity,
                                                int cur, int count) {
  it.c += 2;
  if (it.c < it.wchunks) return;
  it.c = parity;
  it.j = pg_next_slot(it.j, cur, count);
  if (it.j >= 0) return;
  it.t += stride;
  pg_iter_seek(it, tiles, n_tiles, stride, parity, cur, count);
}

__global__ void __launch_bounds__(kPgThreads, 1)
tc_project_gram_kernel(const CUtensorMap* __restrict__ tmaps, const TcTile* __restrict__ tiles, int n_tiles,
                        const MatDesc* __restrict__ mats, const PgMat* __restrict__ pgm, double* __restrict__ part,
                        Ctrl* ctrl) {
  using L = PgSmem;
  constexpr int STAGES = kPgStages;
  extern __shared__ unsigned char tc_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* full_bar = bars;                     // [STAGES] operands landed
  uint64_t* empty_bar = bars + STAGES;           // [STAGES] operands consumed
  uint64_t* tfull_bar = bars + 2 * STAGES;       // [2] accumulator complete
  uint64_t* tempty_bar = bars + 2 * STAGES + 2;  // [2] accumulator drained
  uint64_t* hfull_bar = bars + 2 * STAGES + 4;   // [8 warps][kPgBoxes] history box landed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(hfull_bar + 8 * kPgBoxes);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar + b, 1); mbar_init(tempty_bar + b, 8); }
    for (int s = 0; s < 8 * kPgBoxes; ++s) mbar_init(hfull_bar + s, 1);
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
  const int s_len = mats[0].s;
  const int cur = ring_cur(ctrl, s_len), count = ring_count(ctrl, s_len);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer of the operands
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += stride) {
        const TcTile tile = tiles[t];
        const CUtensorMap* maps = tmaps + tile.mat * kTcMapsPerMat;
        const int n_rem = tile.cols - tile.n0;
        const int n_eff = n_rem >= kPgBN ? kPgBN : n_rem;  // a multiple of 32
        const int nchunks = (n_eff + 63) >> 6;
        const uint32_t bytes = L::kABytes + nchunks * L::kBChunkBytes;
        for (int kb = 0; kb < tile.kblocks; ++kb) {
          if (!mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sA = smem + stage * L::kStageBytes;
          mbar_expect_tx(full_bar + stage, bytes);
          const int k = tile.k0 + kb * kTcBK;
          tma_load_2d(sA, maps + TC_MAP_A_PROJ, k, tile.m0, full_bar + stage);
          for (int c = 0; c < nchunks; ++c)
            tma_load_2d(sA + L::kABytes + c * L::kBChunkBytes, maps + TC_MAP_B_PROJ, tile.n0 + c * 64, k, full_bar + stage);
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
      for (int t = blockIdx.x; t < n_tiles && ok; t += stride, ++local) {
        const TcTile tile = tiles[t];
        const int n_rem = tile.cols - tile.n0;
        const int n_eff = n_rem >= kPgBN ? kPgBN : n_rem;
        const uint32_t idesc = instr_desc(n_eff, false, false);
        const int buf = local & 1;
        const uint32_t tphase = (local >> 1) & 1u;
        if (!mbar_wait(tempty_bar + buf, tphase ^ 1u, abort_flag)) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * kPgBN;
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
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        tc_commit(tfull_bar + buf);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2 .. 9)
    // The two warps of a quarter take the even and the odd 32-column chunks, for R itself and for every older
    // slot alike.  <R, R> and <R, H_j> go through the same function, chunk by chunk in the same order on the same
    // thread (see pg_dot32), so a gradient that repeats bit for bit gives an exactly singular Gram matrix.
    const int quarter = warp & 3;        // TMEM lanes 32 * quarter .. + 31 belong to this warp
    const int parity = (warp - 2) >> 2;
    const int e = warp - 2;
    unsigned char* my_ring = smem + L::kRingOffset + e * kPgBoxes * L::kBoxBytes;
    uint64_t* my_full = hfull_bar + e * kPgBoxes;
    // the box this warp uses next sits in ring position `pos`; `ahead` walks kPgBoxes boxes in front of it
    PgBoxIter ahead;
    ahead.t = blockIdx.x;
    pg_iter_seek(ahead, tiles, n_tiles, stride, parity, cur, count);
    auto issue = [&](int k) {
      // all lanes know the box; lane 0 sends the copy
      if (lane == 0) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the place was just read with plain loads
        mbar_expect_tx(my_full + k, L::kBoxBytes);
        tma_load_2d(my_ring + k * L::kBoxBytes, tmaps + ahead.mat * kTcMapsPerMat + TC_MAP_H_LOAD, ahead.n0 + ahead.c * 32,
                    ahead.j * ahead.rows + ahead.m0 + quarter * 32, my_full + k);
      }
    };
    for (int k = 0; k < kPgBoxes && ahead.valid; ++k) {
      issue(k);
      pg_iter_advance(ahead, tiles, n_tiles, stride, parity, cur, count);
    }
    int pos = 0;
    uint32_t phase = 0;
    int local = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles && ok; t += stride, ++local) {
      const TcTile tile = tiles[t];
      const MatDesc& d = mats[tile.mat];
      const PgMat pm = pgm[tile.mat];
      float* out = d.H + static_cast<long long>(cur) * d.rn;
      const int buf = local & 1;
      const uint32_t tphase = (local >> 1) & 1u;
      const int n_rem = tile.cols - tile.n0;
      const int wchunks = (n_rem >= kPgBN ? kPgBN : n_rem) >> 5;
      const int row = tile.m0 + quarter * 32 + lane;
      const bool row_ok = row < tile.rows;
      float acc[kPgSMax];
#pragma unroll
      for (int j = 0; j < kPgSMax; ++j) acc[j] = 0.f;
      if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar + buf, tphase, abort_flag))) break;
      tc_fence_after();
      const uint32_t tmem_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(buf * kPgBN);
      // first pass over this warp's chunks of the accumulator: write R into the ring slot of this step and
      // sum its squares
      for (int c = parity; c < wchunks; c += 2) {
        uint32_t r[32];
        tc_ld32(tmem_row + static_cast<uint32_t>(c * 32), r);
        tc_wait_ld();
        float4 x[8];
#pragma unroll
        for (int q = 0; q < 8; ++q)
          x[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]),
                             __uint_as_float(r[4 * q + 3]));
        if (row_ok) {
          float4* p = reinterpret_cast<float4*>(out + static_cast<long long>(row) * tile.cols + tile.n0 + c * 32);
#pragma unroll
          for (int q = 0; q < 8; ++q) p[q] = x[q];
          const float tsum = pg_dot32(r, x);
#pragma unroll
          for (int j = 0; j < kPgSMax; ++j)
            if (j == cur) acc[j] += tsum;
        }
      }
      // one pass per older slot: the chunk of R comes back from TMEM for every box (TMEM reads are cheap; holding
      // the whole 256-column row in registers is not possible)
#pragma unroll
      for (int j = 0; j < kPgSMax; ++j) {
        if (j < count && j != cur) {
          for (int c = parity; c < wchunks && ok; c += 2) {
            uint32_t r[32];
            tc_ld32(tmem_row + static_cast<uint32_t>(c * 32), r);
            tc_wait_ld();
            if (!__all_sync(0xffffffffu, mbar_wait(my_full + pos, phase, abort_flag))) {
              ok = false;
            } else {
              // this lane's row of the box: 16-byte piece q sits at piece (q ^ (row & 7)) of the 128-byte row
              const unsigned char* rowp = my_ring + pos * L::kBoxBytes + lane * 128;
              float4 h[8];
#pragma unroll
              for (int q = 0; q < 8; ++q) h[q] = *reinterpret_cast<const float4*>(rowp + ((q ^ (lane & 7)) << 4));
              const float tsum = pg_dot32(r, h);
              if (row_ok) acc[j] += tsum;
              // every lane has read the box: refill its place with the box kPgBoxes further on
              __syncwarp();
              if (ahead.valid) {
                issue(pos);
                pg_iter_advance(ahead, tiles, n_tiles, stride, parity, cur, count);
              }
              if (++pos == kPgBoxes) { pos = 0; phase ^= 1u; }
            }
          }
        }
      }
      // this warp's TMEM reads of the tile are done; with all eight arrivals the MMAs of the tile after next may
      // start (those of the next tile ran into the other buffer meanwhile)
      tc_fence_before();
      if (lane == 0) mbar_arrive(tempty_bar + buf);
      if (!ok) break;
      // this warp's partial row of the tile (zeros for the slots it took no box of)
      const int tile_local = (tile.m0 / kTcBM) * pm.tiles_n + tile.n0 / kPgBN;
      double* prow = part + pm.part_off + (static_cast<long long>(tile_local) * kPgWarpRows + e) * kPgSMax;
#pragma unroll
      for (int j = 0; j < kPgSMax; ++j) {
        const double tj = warp_sum(static_cast<double>(acc[j]));
        if (lane == 0) prow[j] = tj;
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

// One CTA per matrix that took part: add its partial rows (eight groups of threads over disjoint rows, each in a
// fixed order, so the sum is reproducible), then one warp updates row and column `cur` of the raw Gram matrix,
// solves (lambda I + K) w = e_cur and publishes w for the combination tiles of the stream kernel.
__global__ void __launch_bounds__(256) pg_solve_kernel(const MatDesc* __restrict__ mats, const PgMat* __restrict__ pgm,
                                                       const double* __restrict__ part, const int* __restrict__ list,
                                                       const Ctrl* __restrict__ ctrl, const Hyper* __restrict__ hyper) {
  __shared__ double red[8 * 32];
  __shared__ double A[kMaxHistory * (kMaxHistory + 1)];
  const int mat = list[blockIdx.x];
  const MatDesc& d = mats[mat];
  const PgMat pm = pgm[mat];
  const int j = threadIdx.x & 31, g = threadIdx.x >> 5;
  double t0 = 0.0, t1 = 0.0;
  if (j < kPgSMax) {
    const double* base = part + pm.part_off + j;
    const int rows = pm.ntiles * kPgWarpRows;
    int t = g;
    for (; t + 8 < rows; t += 16) {
      t0 += __ldcg(base + static_cast<long long>(t) * kPgSMax);
      t1 += __ldcg(base + static_cast<long long>(t + 8) * kPgSMax);
    }
    if (t < rows) t0 += __ldcg(base + static_cast<long long>(t) * kPgSMax);
  }
  red[g * 32 + j] = t0 + t1;
  __syncthreads();
  if (threadIdx.x < 32) {
    solve_matrix(d, ring_cur(ctrl, d.s), ring_count(ctrl, d.s), hyper->lambda, A, red, 8, 32);
    if (threadIdx.x == 0) {
      __threadfence();
      atomicExch(d.w_ready, ctrl->epoch + 1);
    }
  }
}

inline ngalore_status tc_project_gram_init() {
  if (cudaFuncSetAttribute(tc_project_gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PgSmem::kTotal) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  return NGALORE_OK;
}

}  // namespace ngalore
