// Projection R = P^T G with the new row of the history's Gram matrix formed in its epilogue (Sec. 1; Sec. 2.4:
// y = G^T g, the inner products of the current low-rank gradient with the stacked past ones).
//
// The Gram row needs one read of the whole history ring, which is HBM traffic with no arithmetic to speak of,
// and the projection is tensor-core time with little traffic.  Run one after the other neither hides the other;
// here the old ring slots of the tile an epilogue warp is draining stream through a short shared-memory ring
// (TMA, 128 rows x 32 columns per slot, 128-byte swizzle: the row-per-lane float4 reads are conflict-free) while
// the MMAs of the next tile run into the second accumulator buffer.  Each epilogue thread holds its row of the
// 32-column chunk of R from tcgen05.ld, writes it to the ring slot of the current step and multiplies it into the
// same rows of every older slot.  Products and the per-thread sums over a tile are fp32, everything across
// threads is fp64, as in the stream kernel's Gram pass.  Every epilogue warp writes its partial row per tile
// (no synchronisation between warps); pg_solve_kernel, launched behind this kernel, adds the partial rows of
// a matrix in a fixed order, solves the s x s system and publishes the weights for the combination pass.
//
// Only matrices whose R comes out of a single CTA per tile take part (left projection, K not split, row and
// column counts multiples of 32, 1 <= s <= 16, fp32 history); the others keep the plain projection and the Gram
// tiles of the stream kernel.
//
// Warp roles as in the back-projection: warp 0 TMA producer of the operands, warp 1 TMEM owner and MMA issuer,
// warps 2..9 epilogue (quarter = warp % 4 owns 32 rows; the two warps of a quarter share the history boxes of
// every chunk), warp 10 TMA producer of the history boxes.  Every mbarrier wait is bounded (see mbar_wait).
#pragma once

#include "backproject_tcgen05.cuh"
#include "kernels_stream.cuh"

namespace ngalore {

constexpr int kPgHProducerWarp = 10;
constexpr int kPgThreads = 32 * 11;
// Two operand stages of 48 KB and eight history slots of 16 KB: the kernel is bound by the history stream, which
// wants bytes in flight; the MMAs of a tile take a third of the time its history takes to arrive.
constexpr int kPgStages = 2, kPgSlots = 8;

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

template <int STAGES, int SLOTS>
__global__ void __launch_bounds__(kPgThreads, 1)
tc_project_gram_kernel(const CUtensorMap* __restrict__ tmaps, const TcTile* __restrict__ tiles, int n_tiles,
                       const MatDesc* __restrict__ mats, const PgMat* __restrict__ pgm, double* __restrict__ part,
                       Ctrl* ctrl) {
  using L = BpSmem<STAGES, SLOTS>;
  static_assert(SLOTS % 2 == 0, "the ring is split into two halves");
  constexpr int kHalf = SLOTS / 2;
  extern __shared__ unsigned char tc_smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* full_bar = bars;                     // [STAGES] operands landed
  uint64_t* empty_bar = bars + STAGES;           // [STAGES] operands consumed
  uint64_t* tfull_bar = bars + 2 * STAGES;       // [2] accumulator complete
  uint64_t* tempty_bar = bars + 2 * STAGES + 2;  // [2] accumulator drained
  uint64_t* hfull_bar = bars + 2 * STAGES + 4;   // [SLOTS] history box landed
  uint64_t* hempty_bar = hfull_bar + SLOTS;      // [SLOTS] history box read by its four warps
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(hempty_bar + SLOTS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar + b, 1); mbar_init(tempty_bar + b, 8); }
    for (int s = 0; s < SLOTS; ++s) { mbar_init(hfull_bar + s, 1); mbar_init(hempty_bar + s, 4); }
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
  // ring position and number of gradients held, the same for every matrix of the state
  const int s_len = mats[0].s;
  const int cur = ring_cur(ctrl, s_len), count = ring_count(ctrl, s_len);
  const int n_old = count - 1;  // history boxes per 32-column chunk

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
  } else if (warp == kPgHProducerWarp) {
    // ------------------------------------------------------------------ TMA producer of the history boxes
    // Order: tile, history slot (ascending, the current one left out), 32-column chunk: the boxes of one slot
    // follow each other along the rows, so that DRAM sees 1 KB of a row within a few boxes rather than 128 bytes.
    // The history is one tall matrix of s * lr_rows rows to the tensor map: slot j starts at row j * lr_rows.
    if (lane == 0 && n_old > 0) {
      int pos[2] = {0, 0};           // position inside each half of the ring
      uint32_t phase[2] = {0u, 0u};
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles && ok; t += stride) {
        const TcTile tile = tiles[t];
        const CUtensorMap* mapH = tmaps + tile.mat * kTcMapsPerMat + TC_MAP_H_LOAD;
        const int n_rem = tile.cols - tile.n0;
        const int wchunks = (n_rem >= kPgBN ? kPgBN : n_rem) >> 5;
        for (int j = 0; j < count && ok; ++j) {
          if (j == cur) continue;
          for (int c = 0; c < wchunks; ++c) {
            const int h = c & 1;     // even chunks go through the first half of the ring, odd ones through the second
            const int slot = h * kHalf + pos[h];
            if (!mbar_wait(hempty_bar + slot, phase[h] ^ 1u, abort_flag)) { ok = false; break; }
            mbar_expect_tx(hfull_bar + slot, L::kWSlotBytes);
            tma_load_2d(smem + L::kWOffset + slot * L::kWSlotBytes, mapH, tile.n0 + c * 32, j * tile.rows + tile.m0,
                        hfull_bar + slot);
            if (++pos[h] == kHalf) { pos[h] = 0; phase[h] ^= 1u; }
          }
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
    // slot alike, and each has its own half of the ring (the producer sends a chunk's box to the half of the
    // chunk's parity), so every warp waits for every use of its slots in order, which is what the one phase bit
    // of an mbarrier can tell apart.  The inner products of R with itself and with an older slot go through the
    // same function, chunk by chunk in the same order on the same thread: where a gradient repeats bit for bit,
    // <R, H_j> equals the <H_j, H_j> computed when H_j was new, and the Gram matrix stays exactly singular
    // rather than indefinite by a rounding (lambda then keeps it positive definite).
    const int quarter = warp & 3;        // TMEM lanes 32 * quarter .. + 31 belong to this warp
    const int parity = (warp - 2) >> 2;
    int pos = 0;                         // position inside this warp's half of the ring
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
            const int slot = parity * kHalf + pos;
            if (!__all_sync(0xffffffffu, mbar_wait(hfull_bar + slot, phase, abort_flag))) {
              ok = false;
            } else {
              // this lane's row of the box: 16-byte piece q sits at piece (q ^ (row & 7)) of the 128-byte row
              const unsigned char* rowp =
                  smem + L::kWOffset + slot * L::kWSlotBytes + quarter * L::kWBoxBytes + lane * 128;
              float4 h[8];
#pragma unroll
              for (int q = 0; q < 8; ++q) h[q] = *reinterpret_cast<const float4*>(rowp + ((q ^ (lane & 7)) << 4));
              const float tsum = pg_dot32(r, h);
              if (row_ok) acc[j] += tsum;
              __syncwarp();
              if (lane == 0) mbar_arrive(hempty_bar + slot);
              if (++pos == kHalf) { pos = 0; phase ^= 1u; }
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
      double* prow = part + pm.part_off + (static_cast<long long>(tile_local) * kPgWarpRows + (warp - 2)) * kPgSMax;
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
  if (cudaFuncSetAttribute(tc_project_gram_kernel<kPgStages, kPgSlots>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           BpSmem<kPgStages, kPgSlots>::kTotal) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  return NGALORE_OK;
}

}  // namespace ngalore
