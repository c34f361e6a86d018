// One persistent kernel for the whole history phase of a step: the Gram row of every matrix,
// the s x s solves, and the natural-gradient combination with the Adam moments (Sec. 2.4, 2.2).
//
// Structure: one CTA per SM; a producer warp streams the history (and m, v) through a ring of
// shared-memory stages with bulk asynchronous copies (cp.async.bulk + mbarrier), eight consumer
// warps compute from shared memory.  The producer runs ahead of the consumers across tile and
// matrix boundaries, so the SM always has several stages of loads in flight.
//
// Work items (Gram tiles and combination tiles of all matrices) are fetched in order from a global
// counter by the producer.  Gram items never wait; the CTA that finishes a matrix's last Gram tile
// solves its s x s system and publishes the weights; the consumers of a combination item wait
// (bounded) for that flag.  Every item a combination item depends on sits earlier in the list and
// has been fetched by a CTA that consumes its items in order, so the kernel cannot deadlock.
// All Gram items precede all combination items, so the wait is short except at the very end of the Gram items.
#pragma once

#include <vector>

#include "../../include/ngalore.h"
#include "common.cuh"
#include "gemm_tcgen05.cuh"  // mbarrier wrappers
#include "kernels_stream.cuh"

namespace ngalore {

struct FusedItem {
  int mat;
  int local;
  int kind;  // 0 = Gram tile, 1 = combination tile
  int pad;
};

struct FusedPlan {
  FusedItem* d_items = nullptr;
  int n_items = 0;
  int grid = 0;
  bool hist16 = false;  // the state keeps its history ring in bf16
  bool mom16 = false;   // the state keeps its moments in bf16
};

constexpr long long kSpinLimit = 4000000;  // polls of ~100 ns each before a flag wait is abandoned

struct StageMeta {
  int mat, kind, local, first, last, count;
  int cur, c;  // ring position and number of valid slots of this step (the same for every stage of a launch)
  long long e0;
};

// Stage layout.  fp32 history: SMAX slots of CE floats, then m, then v.  bf16 history (HIST16): SMAX slots of CE
// bf16 values (the current slot's place stays unused), then the current gradient, m and v as floats.
// MOM16: the moments are stored as bf16 (half the bytes of their stages).
template <int SMAX, bool HIST16, bool MOM16 = false>
struct FusedCfg {
  // Elements per stage and slot.  The bf16 history costs more instructions per byte (conversion, two Gram rows),
  // and the per-stage bookkeeping of a consumer thread weighs as much as its arithmetic on two elements, so its
  // stages are twice as long (four elements per thread) even though only two or three of them fit.
  static constexpr int CE = SMAX <= 16 ? (HIST16 ? 2048 : 1024) : 512;
  // consumer threads: the bf16 history costs more instructions per byte (conversion, two Gram rows), so it gets
  // sixteen warps where the registers allow it
  static constexpr int kConsumers = (HIST16 && SMAX <= 16) ? 512 : 256;
  static constexpr int kThreads = kConsumers + 32;
  static constexpr int kHistBytes = SMAX * CE * (HIST16 ? 2 : 4);
  static constexpr int kCurOff = kHistBytes;                          // HIST16: fp32 gradient of this step
  static constexpr int kMOff = kHistBytes + (HIST16 ? CE * 4 : 0);
  static constexpr int kVOff = kMOff + CE * (MOM16 ? 2 : 4);
  static constexpr int kStageBytes = kVOff + CE * (MOM16 ? 2 : 4);
  static constexpr int kStages = HIST16 ? (SMAX <= 8 ? 3 : (SMAX <= 16 ? 2 : 5)) : (SMAX <= 8 ? 5 : 3);
  static constexpr int kBase = kStages * kStageBytes;
  static constexpr int kFullOff = kBase, kEmptyOff = kBase + 64, kMetaOff = kBase + 128, kFlagOff = kBase + 512;
  static constexpr int kWOff = kBase + 640, kRedOff = kBase + 768;
  static constexpr int kRedDoubles = (kConsumers / 32) * SMAX;  // one Gram row per consumer warp
  static constexpr int kAOff = kRedOff + (HIST16 ? 2 : 1) * kRedDoubles * 8;
  static constexpr int kTotal = kAOff + kMaxHistory * (kMaxHistory + 1) * 8;
  static_assert(kStages * sizeof(StageMeta) <= 384, "stage metadata overflows its slot");
  static_assert(kTotal <= 232448, "shared memory budget of one CTA exceeded");
};

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
template <int THREADS>
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) { return __uint_as_float(bits16 << 16); }
__device__ __forceinline__ uint32_t float_to_bf16_bits(float x) {
  return static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(x)));
}

// HIST16: the ring holds bf16 values; the gradient of the current step is read in fp32 from its own buffer
// (MatDesc::H) and its bf16 rounding is written into ring slot `cur` by the combination pass.  The Gram pass
// then also recomputes the row of the slot that was current one step ago, now that it is a rounded value, so
// that Kraw stays the Gram matrix of exactly the values the combination uses.
// MOM16: the moments are read and written as bf16: m rounded to nearest, v rounded stochastically (one step changes
// v by a relative 1 - beta2, less than half a bf16 unit, so rounding to nearest would freeze it) with bits from a
// counter-based generator keyed by (element group, matrix, step index); the direction u of the step comes from
// the unrounded values.
template <int SMAX, bool HIST16, bool MOM16>
__global__ void __launch_bounds__((FusedCfg<SMAX, HIST16, MOM16>::kThreads), 1)
fused_stream_kernel(const MatDesc* __restrict__ mats, const FusedItem* __restrict__ items, int n_items, Ctrl* ctrl,
                    const Hyper* __restrict__ hyper) {
  using C = FusedCfg<SMAX, HIST16, MOM16>;
  constexpr int CE = C::CE;
  constexpr int kConsumerThreads = C::kConsumers;
  constexpr int kGroups = kConsumerThreads / 32;
  constexpr int VEC = CE / kConsumerThreads;  // 4 or 2 elements per thread and stage
  static_assert(VEC == 2 || VEC == 4, "a thread handles two or four elements of a stage");
  extern __shared__ __align__(128) unsigned char fs_smem[];
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(fs_smem + C::kFullOff);
  uint64_t* empty_bar = reinterpret_cast<uint64_t*>(fs_smem + C::kEmptyOff);
  StageMeta* meta = reinterpret_cast<StageMeta*>(fs_smem + C::kMetaOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(fs_smem + C::kFlagOff);
  volatile int* s_flag = abort_flag + 1;
  float* wsm = reinterpret_cast<float*>(fs_smem + C::kWOff);
  double* red = reinterpret_cast<double*>(fs_smem + C::kRedOff);
  double* red2 = red + C::kRedDoubles;  // HIST16 only: the second Gram row
  double* Amat = reinterpret_cast<double*>(fs_smem + C::kAOff);

  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(full_bar + s, 1);
      mbar_init(empty_bar + s, kConsumerThreads / 32);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  const int tag = ctrl->epoch + 1;

  if (tid >= kConsumerThreads) {
    // ------------------------------------------------------------------ producer warp
    // Lane 0 claims items and arms the barriers; every lane issues the bulk copy of "its" slot (lane j copies
    // history slot j, the next two lanes m and v), so a stage's copies are issued in parallel.
    {
      const int lane = tid & 31;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      while (ok) {
        int it = 0;
        if (lane == 0) it = static_cast<int>(atomicAdd(&ctrl->work_counter, 1u));
        it = __shfl_sync(0xffffffffu, it, 0);
        if (it >= n_items) {
          if (lane == 0 && mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag)) {
            meta[stage].kind = -1;
            mbar_arrive(full_bar + stage);
          }
          break;
        }
        const FusedItem item = items[it];
        const MatDesc& d = mats[item.mat];
        const int c = ring_count(ctrl, d.s);
        const int cur_slot = ring_cur(ctrl, d.s);
        const int ncopies = c + (item.kind == 1 ? 2 : 0);
        const long long e0 = static_cast<long long>(item.local) * d.te;
        const long long e1 = (e0 + d.te < d.rn) ? e0 + d.te : d.rn;
        for (long long e = e0; e < e1; e += CE) {
          const int cnt = (e1 - e < CE) ? static_cast<int>(e1 - e) : CE;
          int good = 1;
          if (lane == 0) good = mbar_wait(empty_bar + stage, phase ^ 1u, abort_flag) ? 1 : 0;
          good = __shfl_sync(0xffffffffu, good, 0);
          if (!good) { ok = false; break; }
          unsigned char* sb = fs_smem + stage * C::kStageBytes;
          const uint32_t bytes = static_cast<uint32_t>(cnt) * 4u;
          if (lane == 0) {
            StageMeta mt;
            mt.mat = item.mat; mt.kind = item.kind; mt.local = item.local;
            mt.first = (e == e0) ? 1 : 0; mt.last = (e + CE >= e1) ? 1 : 0; mt.count = cnt; mt.e0 = e;
            mt.cur = cur_slot; mt.c = c;
            meta[stage] = mt;
            const uint32_t hist_bytes = HIST16 ? bytes * static_cast<uint32_t>(c) - (bytes / 2) * static_cast<uint32_t>(c - 1)
                                               : bytes * static_cast<uint32_t>(c);
            const uint32_t mom_bytes = item.kind == 1 ? (MOM16 ? bytes : 2u * bytes) : 0u;
            mbar_expect_tx(full_bar + stage, hist_bytes + mom_bytes);
          }
          __syncwarp();
          for (int j = lane; j < ncopies; j += 32) {
            if (j < c) {
              if (!HIST16)
                bulk_load(sb + j * CE * 4, d.H + static_cast<long long>(j) * d.rn + e, bytes, full_bar + stage);
              else if (j == cur_slot)
                bulk_load(sb + C::kCurOff, d.H + e, bytes, full_bar + stage);
              else
                bulk_load(sb + j * CE * 2, d.H16 + static_cast<long long>(j) * d.rn + e, bytes / 2, full_bar + stage);
            } else {
              const int k = j - c;  // 0: m, 1: v
              if (MOM16)
                bulk_load(sb + (k == 0 ? C::kMOff : C::kVOff), (k == 0 ? d.m16 : d.v16) + e, bytes / 2, full_bar + stage);
              else
                bulk_load(sb + (k == 0 ? C::kMOff : C::kVOff), (k == 0 ? d.m : d.v) + e, bytes, full_bar + stage);
            }
          }
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers (8 or 16 warps)
    const int warp = tid >> 5, lane = tid & 31;
    const Hyper hp = *hyper;
    int stage = 0;
    uint32_t phase = 0;
    float acc[SMAX];
    float acc2[HIST16 ? SMAX : 1];  // HIST16: inner products with the slot that was current one step ago
    float w[SMAX];
#pragma unroll
    for (int j = 0; j < SMAX; ++j) { acc[j] = 0.f; w[j] = 0.f; }
#pragma unroll
    for (int j = 0; j < (HIST16 ? SMAX : 1); ++j) acc2[j] = 0.f;
    bool item_bad = false, item_ok = true;
    // per-item pointers of the combination pass, fetched once at the item's first stage
    float *it_m = nullptr, *it_v = nullptr, *it_cur = nullptr;
    __half* it_u = nullptr;
    uint16_t *it_h16 = nullptr, *it_m16 = nullptr, *it_v16 = nullptr;
    unsigned int it_mat = 0, it_step = 0;
    while (true) {
      if (!mbar_wait(full_bar + stage, phase, abort_flag)) break;
      const StageMeta mt = meta[stage];
      if (mt.kind < 0) break;
      const MatDesc& d = mats[mt.mat];
      const int cur = mt.cur, c = mt.c;
      const unsigned char* sbytes = fs_smem + stage * C::kStageBytes;
      const int idx = tid * VEC;
      // this thread's VEC elements of history slot j in this stage
      auto load_hist = [&](int j, float (&h)[VEC]) {
        if (!HIST16) {
          const float* p = reinterpret_cast<const float*>(sbytes) + j * CE + idx;
#pragma unroll
          for (int q = 0; q < VEC; ++q) h[q] = p[q];
        } else if (j == cur) {
          const float* p = reinterpret_cast<const float*>(sbytes + C::kCurOff) + idx;
#pragma unroll
          for (int q = 0; q < VEC; ++q) h[q] = p[q];
        } else {
          const uint32_t* p = reinterpret_cast<const uint32_t*>(sbytes + (j * CE + idx) * 2);
#pragma unroll
          for (int q = 0; q < VEC; q += 2) {
            const uint32_t pair = p[q >> 1];
            h[q] = bf16_bits_to_float(pair & 0xFFFFu);
            h[q + 1] = bf16_bits_to_float(pair >> 16);
          }
        }
      };
      // this thread's VEC elements of a moment in this stage
      auto load_moment = [&](int off, float (&x)[VEC]) {
        if (!MOM16) {
          const float* p = reinterpret_cast<const float*>(sbytes + off) + idx;
#pragma unroll
          for (int q = 0; q < VEC; ++q) x[q] = p[q];
        } else {
          const uint32_t* p = reinterpret_cast<const uint32_t*>(sbytes + off + idx * 2);
#pragma unroll
          for (int q = 0; q < VEC; q += 2) {
            const uint32_t pair = p[q >> 1];
            x[q] = bf16_bits_to_float(pair & 0xFFFFu);
            x[q + 1] = bf16_bits_to_float(pair >> 16);
          }
        }
      };
      const bool two_rows = HIST16 && c >= 2;
      const int prev = two_rows ? (cur == 0 ? d.s : cur) - 1 : 0;
      if (mt.kind == 0) {
        if (mt.first) {
#pragma unroll
          for (int j = 0; j < SMAX; ++j) acc[j] = 0.f;
#pragma unroll
          for (int j = 0; j < (HIST16 ? SMAX : 1); ++j) acc2[j] = 0.f;
        }
        if (idx < mt.count) {
          float x[VEC], xp[VEC];
          load_hist(cur, x);
          if (two_rows) load_hist(prev, xp);
#pragma unroll
          for (int j = 0; j < SMAX; ++j) {
            if (j < c) {
              float h[VEC];
              load_hist(j, h);
              float t = 0.f;
#pragma unroll
              for (int q = 0; q < VEC; ++q) t += x[q] * h[q];
              acc[j] += t;
              if (HIST16 && two_rows) {
                float t2 = 0.f;
#pragma unroll
                for (int q = 0; q < VEC; ++q) t2 += xp[q] * h[q];
                acc2[HIST16 ? j : 0] += t2;
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar + stage);
        if (mt.last) {
#pragma unroll
          for (int j = 0; j < SMAX; ++j) {
            const double t = warp_sum(static_cast<double>(acc[j]));
            if (lane == 0) red[warp * SMAX + j] = t;
            if (HIST16) {
              const double t2 = warp_sum(static_cast<double>(acc2[HIST16 ? j : 0]));
              if (lane == 0) red2[warp * SMAX + j] = t2;
            }
          }
          consumer_sync<kConsumerThreads>();
          // per-tile partial rows: [tile][s] (fp32 history) or [tile][2][s] (HIST16: row of `cur`, row of `prev`)
          constexpr int kRows = HIST16 ? 2 : 1;
          if (tid < kRows * 32 && (tid & 31) < SMAX && (tid & 31) < d.s) {
            const int row = tid >> 5, j = tid & 31;
            const double* src = row == 0 ? red : red2;
            double t = 0.0;
#pragma unroll
            for (int ww = 0; ww < kConsumerThreads / 32; ++ww) t += src[ww * SMAX + j];
            d.gpart[(static_cast<long long>(mt.local) * kRows + row) * d.s + j] = t;
            __threadfence();
          }
          consumer_sync<kConsumerThreads>();
          if (tid == 0) {
            const int done = atomicAdd(d.gram_done, 1);
            *s_flag = (done == d.ntiles - 1) ? 1 : 0;
          }
          consumer_sync<kConsumerThreads>();
          if (*s_flag) {
            // last Gram tile of this matrix: all consumers pre-sum the per-tile partials (fixed partition,
            // so the result is reproducible), then one warp factors and solves
            __threadfence();
            const int j = tid & 31, g = tid >> 5;
            if (j < SMAX) {
#pragma unroll
              for (int row = 0; row < kRows; ++row) {
                double t0 = 0.0, t1 = 0.0;
                if (j < d.s) {
                  const double* gp = d.gpart + static_cast<long long>(row) * d.s + j;
                  const long long tstride = static_cast<long long>(kRows) * d.s;
                  int t = g;
                  for (; t + kGroups < d.ntiles; t += 2 * kGroups) {
                    t0 += __ldcg(gp + t * tstride);
                    t1 += __ldcg(gp + (t + kGroups) * tstride);
                  }
                  if (t < d.ntiles) t0 += __ldcg(gp + t * tstride);
                }
                (row == 0 ? red : red2)[g * SMAX + j] = t0 + t1;
              }
            }
            consumer_sync<kConsumerThreads>();
            if (tid < 32) {
              if (two_rows) {
                // row and column `prev` of Kraw against the stored (rounded) values; its entry with `cur`
                // is written with the rest of row `cur` below, from the same products
                double rowp = 0.0;
                if (tid < c && tid != cur) {
                  for (int gg = 0; gg < kConsumerThreads / 32; ++gg) rowp += red2[gg * SMAX + tid];
                  if (isfinite(rowp)) {
                    d.Kraw[prev * d.s + tid] = rowp;
                    d.Kraw[tid * d.s + prev] = rowp;
                  }
                }
                __syncwarp();
              }
              solve_matrix(d, cur, c, hp.lambda, Amat, red, kConsumerThreads / 32, SMAX);
              if (tid == 0) {
                *d.gram_done = 0;
                __threadfence();
                if (ctrl->debug_withhold != mt.mat + 1) atomicExch(d.w_ready, tag);
              }
            }
          }
          consumer_sync<kConsumerThreads>();
        }
      } else {
        if (mt.first) {
          item_ok = true;
          if (d.s > 0) {
            if (tid == 0) {
              const volatile int* flag = d.w_ready;
              const long long limit = ctrl->spin_limit > 0 ? ctrl->spin_limit : kSpinLimit;
              long long spins = 0;
              int ok = 1;
              while (*flag != tag) {
                if (++spins > limit) { ok = 0; break; }
                __nanosleep(100);
              }
              if (!ok) {
                // The weights never came: this matrix takes no update in this step (the back-projection skips it)
                // and says why.  Tiles of it that other CTAs did combine have advanced their part of m and v.
                atomicExch(&ctrl->timeout_flag, 1);
                atomicExch(d.step_bad, 1);
                atomicCAS(d.status, 0, 8 /* NGALORE_ERR_TIMEOUT */);
              }
              *s_flag = ok;
            }
            consumer_sync<kConsumerThreads>();
            item_ok = *s_flag != 0;
            __threadfence();
          }
          if (tid < kMaxHistory) wsm[tid] = __ldcg(d.wsol + tid);
          item_bad = __ldcg(d.step_bad) != 0;
          it_m = d.m; it_v = d.v; it_u = d.u16;
          it_m16 = d.m16; it_v16 = d.v16;
          it_mat = static_cast<unsigned int>(d.index);
          it_step = static_cast<unsigned int>(ctrl->k);
          it_cur = current_gradient(d, cur);
          it_h16 = HIST16 ? d.H16 + static_cast<long long>(cur) * d.rn : nullptr;
          consumer_sync<kConsumerThreads>();
#pragma unroll
          for (int j = 0; j < SMAX; ++j) w[j] = wsm[j];
        }
        if (item_ok && idx < mt.count) {
          const long long e = mt.e0 + idx;
          if (item_bad) {
            // The poisoned slot becomes a zero gradient; m, v are left alone and the update is zero.
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
              it_cur[e + q] = 0.f;
              it_u[e + q] = __float2half_rn(0.f);
              if (HIST16) it_h16[e + q] = 0;
            }
          } else {
            float n[VEC], mm[VEC], vv[VEC], uu[VEC];
#pragma unroll
            for (int q = 0; q < VEC; ++q) n[q] = 0.f;
#pragma unroll
            for (int j = 0; j < SMAX; ++j) {
              if (j < c) {
                float h[VEC];
                load_hist(j, h);
#pragma unroll
                for (int q = 0; q < VEC; ++q) n[q] = fmaf(w[j], h[q], n[q]);
              }
            }
            if (HIST16) {
              // from the next step on this gradient is an old one: store its bf16 rounding in the ring
              float x[VEC];
              load_hist(cur, x);
              uint32_t* dst = reinterpret_cast<uint32_t*>(it_h16 + e);
#pragma unroll
              for (int q = 0; q < VEC; q += 2) dst[q >> 1] = float_to_bf16_bits(x[q]) | (float_to_bf16_bits(x[q + 1]) << 16);
            }
            load_moment(C::kMOff, mm);
            load_moment(C::kVOff, vv);
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
              mm[q] = hp.beta1 * mm[q] + (1.f - hp.beta1) * n[q];
              vv[q] = hp.beta2 * vv[q] + (1.f - hp.beta2) * n[q] * n[q];
              uu[q] = mm[q] / sqrtf(vv[q] + hp.eps);
            }
            if (MOM16) {
              // elements 4 g .. 4 g + 3 take the upper halves of the four words of one generator call
              uint32_t* dm = reinterpret_cast<uint32_t*>(it_m16 + e);
              uint32_t* dv = reinterpret_cast<uint32_t*>(it_v16 + e);
#pragma unroll
              for (int q0 = 0; q0 < VEC; q0 += 4) {
                const unsigned long long grp = static_cast<unsigned long long>(e + q0) >> 2;
                const uint4 rnd = philox4x32_10(make_uint4(static_cast<unsigned int>(grp), static_cast<unsigned int>(grp >> 32),
                                                           it_mat, it_step), hp.seed_lo, hp.seed_hi);
                const unsigned int rb[4] = {rnd.x >> 16, rnd.y >> 16, rnd.z >> 16, rnd.w >> 16};
#pragma unroll
                for (int q = q0; q < q0 + 4 && q < VEC; q += 2) {
                  // (VEC = 2: e is a multiple of 2, the pair is words 0, 1 or words 2, 3 of its group)
                  const int w0 = VEC == 2 ? static_cast<int>(e & 2) : q - q0;
                  dm[q >> 1] = float_to_bf16_bits(mm[q]) | (float_to_bf16_bits(mm[q + 1]) << 16);
                  dv[q >> 1] = stochastic_bf16_bits(vv[q], rb[w0]) | (stochastic_bf16_bits(vv[q + 1], rb[w0 + 1]) << 16);
                }
              }
              if (VEC == 4) *reinterpret_cast<uint2*>(it_u + e) = pack_f16x4(uu[0], uu[1], uu[2 % VEC], uu[3 % VEC]);
              else *reinterpret_cast<uint32_t*>(it_u + e) = pack_f16x4(uu[0], uu[1], 0.f, 0.f).x;
            } else if (VEC == 4) {
              *reinterpret_cast<float4*>(it_m + e) = make_float4(mm[0], mm[1], mm[2 % VEC], mm[3 % VEC]);
              *reinterpret_cast<float4*>(it_v + e) = make_float4(vv[0], vv[1], vv[2 % VEC], vv[3 % VEC]);
              *reinterpret_cast<uint2*>(it_u + e) = pack_f16x4(uu[0], uu[1], uu[2 % VEC], uu[3 % VEC]);
            } else {
              *reinterpret_cast<float2*>(it_m + e) = make_float2(mm[0], mm[1]);
              *reinterpret_cast<float2*>(it_v + e) = make_float2(vv[0], vv[1]);
              *reinterpret_cast<uint32_t*>(it_u + e) = pack_f16x4(uu[0], uu[1], 0.f, 0.f).x;
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar + stage);
      }
      if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
    }
  }
  __syncthreads();
  if (*abort_flag) {
    // a wait ran out: give bulk copies that may still be in flight time to land before the CTA retires
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
    if (tid == 0) atomicExch(&ctrl->timeout_flag, 1);
  }
}

template <int SMAX, bool HIST16, bool MOM16>
inline cudaError_t fused_set_smem() {
  return cudaFuncSetAttribute(fused_stream_kernel<SMAX, HIST16, MOM16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              FusedCfg<SMAX, HIST16, MOM16>::kTotal);
}

template <bool HIST16, bool MOM16>
inline cudaError_t fused_set_smem_for(int s) {
  return s <= 8 ? fused_set_smem<8, HIST16, MOM16>() : (s <= 16 ? fused_set_smem<16, HIST16, MOM16>() : fused_set_smem<32, HIST16, MOM16>());
}

// skip_gram (optional, one entry per matrix): 1 where the Gram row and the solve of a matrix are done before this
// kernel runs (projection with the Gram row in its epilogue); such a matrix gets combination tiles only.
inline ngalore_status fused_plan_create(FusedPlan& plan, const std::vector<MatDesc>& mats, int s, int sm_count,
                                        const std::vector<int>* skip_gram = nullptr) {
  plan.grid = sm_count;
  // Item order: every Gram tile (matrix order), then every combination tile (same order).  A CTA that picks
  // up a combination tile then never waits for a Gram tile that is still running, except for the last few
  // matrices.  Measured against keeping a matrix's combination pass close behind its Gram pass (in the hope
  // of L2 hits on its history): the stalls of the close order cost far more than the hits gain; on the 1.1B
  // shapes the phase went from 4.85 ms to 4.2 ms, on the 130M shapes from 0.51 ms to 0.35 ms.
  std::vector<FusedItem> items;
  const int n = static_cast<int>(mats.size());
  for (int i = 0; i < n; ++i) {
    if (mats[i].s == 0) continue;
    if (skip_gram != nullptr && (*skip_gram)[i]) continue;
    for (int t = 0; t < mats[i].ntiles; ++t) items.push_back(FusedItem{i, t, 0, 0});
  }
  for (int i = 0; i < n; ++i)
    for (int t = 0; t < mats[i].ntiles; ++t) items.push_back(FusedItem{i, t, 1, 0});
  plan.n_items = static_cast<int>(items.size());
  if (plan.grid > plan.n_items) plan.grid = plan.n_items;
  if (cudaMalloc(&plan.d_items, sizeof(FusedItem) * items.size()) != cudaSuccess) {
    plan.d_items = nullptr;
    return NGALORE_ERR_ALLOC;
  }
  if (cudaMemcpy(plan.d_items, items.data(), sizeof(FusedItem) * items.size(), cudaMemcpyHostToDevice) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  plan.hist16 = !mats.empty() && mats[0].H16 != nullptr;
  plan.mom16 = !mats.empty() && mats[0].m16 != nullptr;
  const cudaError_t e = plan.hist16 ? (plan.mom16 ? fused_set_smem_for<true, true>(s) : fused_set_smem_for<true, false>(s))
                                    : (plan.mom16 ? fused_set_smem_for<false, true>(s) : fused_set_smem_for<false, false>(s));
  return e == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

inline void fused_plan_destroy(FusedPlan& plan) {
  if (plan.d_items) cudaFree(plan.d_items);
  plan.d_items = nullptr;
}

template <int SMAX, bool HIST16, bool MOM16>
inline void fused_launch_one(const FusedPlan& plan, const MatDesc* d_mats, Ctrl* d_ctrl, const Hyper* d_hyper,
                             cudaStream_t stream) {
  using C = FusedCfg<SMAX, HIST16, MOM16>;
  fused_stream_kernel<SMAX, HIST16, MOM16><<<plan.grid, C::kThreads, C::kTotal, stream>>>(d_mats, plan.d_items, plan.n_items,
                                                                                         d_ctrl, d_hyper);
}

template <bool HIST16, bool MOM16>
inline void fused_launch_for(const FusedPlan& plan, const MatDesc* d_mats, Ctrl* d_ctrl, const Hyper* d_hyper, int s,
                             cudaStream_t stream) {
  if (s <= 8) fused_launch_one<8, HIST16, MOM16>(plan, d_mats, d_ctrl, d_hyper, stream);
  else if (s <= 16) fused_launch_one<16, HIST16, MOM16>(plan, d_mats, d_ctrl, d_hyper, stream);
  else fused_launch_one<32, HIST16, MOM16>(plan, d_mats, d_ctrl, d_hyper, stream);
}

inline ngalore_status fused_stream_launch(FusedPlan& plan, const MatDesc* d_mats, int /*n_mats*/, Ctrl* d_ctrl,
                                          const Hyper* d_hyper, int s, cudaStream_t stream, int64_t* launches) {
  if (plan.hist16) {
    if (plan.mom16) fused_launch_for<true, true>(plan, d_mats, d_ctrl, d_hyper, s, stream);
    else fused_launch_for<true, false>(plan, d_mats, d_ctrl, d_hyper, s, stream);
  } else {
    if (plan.mom16) fused_launch_for<false, true>(plan, d_mats, d_ctrl, d_hyper, s, stream);
    else fused_launch_for<false, false>(plan, d_mats, d_ctrl, d_hyper, s, stream);
  }
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

}  // namespace ngalore
