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
};

constexpr long long kSpinLimit = 4000000;  // polls of ~100 ns each before a flag wait is abandoned
constexpr int kConsumerThreads = 256;
constexpr int kFusedThreads = kConsumerThreads + 32;

struct StageMeta {
  int mat, kind, local, first, last, count;
  long long e0;
};

template <int SMAX>
struct FusedCfg {
  static constexpr int CE = SMAX <= 16 ? 1024 : 512;  // elements per stage and slot
  static constexpr int kSlots = SMAX + 2;             // history slots + m + v
  static constexpr int kStageBytes = kSlots * CE * 4;
  static constexpr int kStages = SMAX <= 8 ? 5 : 3;
  static constexpr int kBase = kStages * kStageBytes;
  static constexpr int kFullOff = kBase, kEmptyOff = kBase + 64, kMetaOff = kBase + 128, kFlagOff = kBase + 384;
  static constexpr int kWOff = kBase + 512, kRedOff = kBase + 640;
  static constexpr int kAOff = kRedOff + (kConsumerThreads / 32) * SMAX * 8;
  static constexpr int kTotal = kAOff + kMaxHistory * (kMaxHistory + 1) * 8;
  static_assert(kStages * sizeof(StageMeta) <= 256, "stage metadata overflows its slot");
  static_assert(kTotal <= 232448, "shared memory budget of one CTA exceeded");
};

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
}

template <int SMAX>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_stream_kernel(const MatDesc* __restrict__ mats, const FusedItem* __restrict__ items, int n_items, Ctrl* ctrl,
                    const Hyper* __restrict__ hyper) {
  using C = FusedCfg<SMAX>;
  constexpr int CE = C::CE;
  constexpr int VEC = CE / kConsumerThreads;  // 4 or 2 elements per thread and stage
  extern __shared__ __align__(128) unsigned char fs_smem[];
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(fs_smem + C::kFullOff);
  uint64_t* empty_bar = reinterpret_cast<uint64_t*>(fs_smem + C::kEmptyOff);
  StageMeta* meta = reinterpret_cast<StageMeta*>(fs_smem + C::kMetaOff);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(fs_smem + C::kFlagOff);
  volatile int* s_flag = abort_flag + 1;
  float* wsm = reinterpret_cast<float*>(fs_smem + C::kWOff);
  double* red = reinterpret_cast<double*>(fs_smem + C::kRedOff);
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
            meta[stage] = mt;
            mbar_expect_tx(full_bar + stage, bytes * static_cast<uint32_t>(ncopies));
          }
          __syncwarp();
          for (int j = lane; j < ncopies; j += 32) {
            if (j < c) {
              bulk_load(sb + j * CE * 4, d.H + static_cast<long long>(j) * d.rn + e, bytes, full_bar + stage);
            } else {
              const int k = j - c;  // 0: m, 1: v
              bulk_load(sb + (SMAX + k) * CE * 4, (k == 0 ? d.m : d.v) + e, bytes, full_bar + stage);
            }
          }
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumers (256 threads)
    const int warp = tid >> 5, lane = tid & 31;
    const Hyper hp = *hyper;
    int stage = 0;
    uint32_t phase = 0;
    float acc[SMAX];
    float w[SMAX];
#pragma unroll
    for (int j = 0; j < SMAX; ++j) { acc[j] = 0.f; w[j] = 0.f; }
    bool item_bad = false, item_ok = true;
    while (true) {
      if (!mbar_wait(full_bar + stage, phase, abort_flag)) break;
      const StageMeta mt = meta[stage];
      if (mt.kind < 0) break;
      const MatDesc& d = mats[mt.mat];
      const int cur = ring_cur(ctrl, d.s), c = ring_count(ctrl, d.s);
      const float* sb = reinterpret_cast<const float*>(fs_smem + stage * C::kStageBytes);
      const int idx = tid * VEC;
      if (mt.kind == 0) {
        if (mt.first) {
#pragma unroll
          for (int j = 0; j < SMAX; ++j) acc[j] = 0.f;
        }
        if (idx < mt.count) {
          float x[VEC];
#pragma unroll
          for (int q = 0; q < VEC; ++q) x[q] = sb[cur * CE + idx + q];
#pragma unroll
          for (int j = 0; j < SMAX; ++j) {
            if (j < c) {
              float t = 0.f;
#pragma unroll
              for (int q = 0; q < VEC; ++q) t += x[q] * sb[j * CE + idx + q];
              acc[j] += t;
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
          }
          consumer_sync();
          if (tid < SMAX && tid < d.s) {
            double t = 0.0;
#pragma unroll
            for (int ww = 0; ww < kConsumerThreads / 32; ++ww) t += red[ww * SMAX + tid];
            d.gpart[static_cast<long long>(mt.local) * d.s + tid] = t;
            __threadfence();
          }
          consumer_sync();
          if (tid == 0) {
            const int done = atomicAdd(d.gram_done, 1);
            *s_flag = (done == d.ntiles - 1) ? 1 : 0;
          }
          consumer_sync();
          if (*s_flag) {
            // last Gram tile of this matrix: all consumers pre-sum the per-tile partials (fixed partition,
            // so the result is reproducible), then one warp factors and solves
            __threadfence();
            const int j = tid & 31, g = tid >> 5;
            if (j < SMAX) {
              double t0 = 0.0, t1 = 0.0;
              if (j < d.s) {
                int t = g;
                for (; t + 8 < d.ntiles; t += 16) {
                  t0 += __ldcg(d.gpart + static_cast<long long>(t) * d.s + j);
                  t1 += __ldcg(d.gpart + static_cast<long long>(t + 8) * d.s + j);
                }
                if (t < d.ntiles) t0 += __ldcg(d.gpart + static_cast<long long>(t) * d.s + j);
              }
              red[g * SMAX + j] = t0 + t1;
            }
            consumer_sync();
            if (tid < 32) {
              solve_matrix(d, cur, c, hp.lambda, Amat, red, kConsumerThreads / 32, SMAX);
              if (tid == 0) {
                *d.gram_done = 0;
                __threadfence();
                atomicExch(d.w_ready, tag);
              }
            }
          }
          consumer_sync();
        }
      } else {
        if (mt.first) {
          item_ok = true;
          if (d.s > 0) {
            if (tid == 0) {
              const volatile int* flag = d.w_ready;
              long long spins = 0;
              int ok = 1;
              while (*flag != tag) {
                if (++spins > kSpinLimit) { ok = 0; break; }
                __nanosleep(100);
              }
              if (!ok) atomicExch(&ctrl->timeout_flag, 1);
              *s_flag = ok;
            }
            consumer_sync();
            item_ok = *s_flag != 0;
            __threadfence();
          }
          if (tid < kMaxHistory) wsm[tid] = __ldcg(d.wsol + tid);
          item_bad = __ldcg(d.step_bad) != 0;
          consumer_sync();
#pragma unroll
          for (int j = 0; j < SMAX; ++j) w[j] = wsm[j];
        }
        if (item_ok && idx < mt.count) {
          const long long e = mt.e0 + idx;
          if (item_bad) {
            // The poisoned slot becomes a zero gradient; m, v are left alone and the update is zero.
            float* Hc = d.H + static_cast<long long>(cur) * d.rn + e;
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
              Hc[q] = 0.f;
              d.u16[e + q] = __float2half_rn(0.f);
            }
          } else {
            float n[VEC], mm[VEC], vv[VEC], uu[VEC];
#pragma unroll
            for (int q = 0; q < VEC; ++q) n[q] = 0.f;
#pragma unroll
            for (int j = 0; j < SMAX; ++j) {
              if (j < c) {
#pragma unroll
                for (int q = 0; q < VEC; ++q) n[q] = fmaf(w[j], sb[j * CE + idx + q], n[q]);
              }
            }
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
              mm[q] = hp.beta1 * sb[SMAX * CE + idx + q] + (1.f - hp.beta1) * n[q];
              vv[q] = hp.beta2 * sb[(SMAX + 1) * CE + idx + q] + (1.f - hp.beta2) * n[q] * n[q];
              uu[q] = mm[q] / sqrtf(vv[q] + hp.eps);
            }
            if (VEC == 4) {
              *reinterpret_cast<float4*>(d.m + e) = make_float4(mm[0], mm[1], mm[2 % VEC], mm[3 % VEC]);
              *reinterpret_cast<float4*>(d.v + e) = make_float4(vv[0], vv[1], vv[2 % VEC], vv[3 % VEC]);
              *reinterpret_cast<uint2*>(d.u16 + e) = pack_f16x4(uu[0], uu[1], uu[2 % VEC], uu[3 % VEC]);
            } else {
              *reinterpret_cast<float2*>(d.m + e) = make_float2(mm[0], mm[1]);
              *reinterpret_cast<float2*>(d.v + e) = make_float2(vv[0], vv[1]);
              *reinterpret_cast<uint32_t*>(d.u16 + e) = pack_f16x4(uu[0], uu[1], 0.f, 0.f).x;
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

inline ngalore_status fused_plan_create(FusedPlan& plan, const std::vector<MatDesc>& mats, int s, int sm_count) {
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
  cudaError_t e;
  if (s <= 8)
    e = cudaFuncSetAttribute(fused_stream_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, FusedCfg<8>::kTotal);
  else if (s <= 16)
    e = cudaFuncSetAttribute(fused_stream_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, FusedCfg<16>::kTotal);
  else
    e = cudaFuncSetAttribute(fused_stream_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, FusedCfg<32>::kTotal);
  return e == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

inline void fused_plan_destroy(FusedPlan& plan) {
  if (plan.d_items) cudaFree(plan.d_items);
  plan.d_items = nullptr;
}

inline ngalore_status fused_stream_launch(FusedPlan& plan, const MatDesc* d_mats, int /*n_mats*/, Ctrl* d_ctrl,
                                          const Hyper* d_hyper, int s, cudaStream_t stream, int64_t* launches) {
  if (s <= 8)
    fused_stream_kernel<8><<<plan.grid, kFusedThreads, FusedCfg<8>::kTotal, stream>>>(d_mats, plan.d_items, plan.n_items, d_ctrl, d_hyper);
  else if (s <= 16)
    fused_stream_kernel<16><<<plan.grid, kFusedThreads, FusedCfg<16>::kTotal, stream>>>(d_mats, plan.d_items, plan.n_items, d_ctrl, d_hyper);
  else
    fused_stream_kernel<32><<<plan.grid, kFusedThreads, FusedCfg<32>::kTotal, stream>>>(d_mats, plan.d_items, plan.n_items, d_ctrl, d_hyper);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

}  // namespace ngalore
