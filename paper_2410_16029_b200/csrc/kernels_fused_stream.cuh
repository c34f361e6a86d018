// One persistent kernel for the whole history phase of a step: the Gram row of every matrix,
// the s x s solves, and the natural-gradient combination with the Adam moments (Sec. 2.4, 2.2).
//
// Work items are fetched in order from a global counter.  Gram items never wait; the CTA that
// finishes a matrix's last Gram tile solves its s x s system and publishes the weights; combination
// items wait (bounded) for that flag.  Every item a combination item depends on sits earlier in
// the list and has therefore been fetched by a running CTA, so the kernel cannot deadlock whatever
// the grid size.  The list interleaves matrices so that the combination pass of a matrix starts
// while its history is still in L2 and the wait is hidden behind the next matrix's Gram tiles.
#pragma once

#include <vector>

#include "../../include/ngalore.h"
#include "common.cuh"
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
  int tile_elems = 0;
};

constexpr long long kSpinLimit = 4000000;  // polls of ~100 ns each before a wait is abandoned

template <int SMAX>
__global__ void __launch_bounds__(kStreamThreads, 2)
fused_stream_kernel(const MatDesc* __restrict__ mats, const FusedItem* __restrict__ items, int n_items, Ctrl* ctrl,
                    const Hyper* __restrict__ hyper, int tile_elems) {
  __shared__ double red[(kStreamThreads / 32) * SMAX];
  __shared__ double A[kMaxHistory * (kMaxHistory + 1)];
  __shared__ float wsm[kMaxHistory];
  __shared__ int s_item, s_flag;
  const int tid = threadIdx.x;
  const int tag = ctrl->epoch + 1;
  const Hyper hp = *hyper;
  while (true) {
    if (tid == 0) s_item = static_cast<int>(atomicAdd(&ctrl->work_counter, 1u));
    __syncthreads();
    const int it = s_item;
    __syncthreads();
    if (it >= n_items) break;
    const FusedItem item = items[it];
    const MatDesc& d = mats[item.mat];
    const int cur = ring_cur(ctrl, d.s), c = ring_count(ctrl, d.s);
    if (item.kind == 0) {
      gram_tile<SMAX>(d, item.local, cur, c, tile_elems, red);
      if (tid == 0) {
        __threadfence();
        const int done = atomicAdd(d.gram_done, 1);
        s_flag = (done == d.ntiles - 1) ? 1 : 0;
      }
      __syncthreads();
      if (s_flag && tid < 32) {
        __threadfence();
        solve_matrix(d, cur, c, hp.lambda, A);
        if (tid == 0) {
          *d.gram_done = 0;
          __threadfence();
          atomicExch(d.w_ready, tag);
        }
      }
      __syncthreads();
    } else {
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
          s_flag = ok;
        }
        __syncthreads();
        const int ok = s_flag;
        __syncthreads();
        if (!ok) continue;
        __threadfence();
      }
      if (tid < kMaxHistory) wsm[tid] = __ldcg(d.wsol + tid);
      __syncthreads();
      combine_tile<SMAX>(d, item.local, cur, c, tile_elems, hp, wsm);
      __syncthreads();
    }
  }
}

inline ngalore_status fused_plan_create(FusedPlan& plan, const std::vector<MatDesc>& mats, int tile_elems, int sm_count) {
  plan.tile_elems = tile_elems;
  plan.grid = sm_count * 2;
  const int head = plan.grid * 2;  // Gram tiles of the next matrix issued before a matrix's combination pass
  std::vector<FusedItem> items;
  const int n = static_cast<int>(mats.size());
  auto gram_range = [&](int i, int t0, int t1) {
    if (mats[i].s == 0) return;
    for (int t = t0; t < t1; ++t) items.push_back(FusedItem{i, t, 0, 0});
  };
  auto combine_all = [&](int i) {
    // reverse order: the tiles read last by the Gram pass are the most likely to be in L2 still
    for (int t = mats[i].ntiles - 1; t >= 0; --t) items.push_back(FusedItem{i, t, 1, 0});
  };
  for (int i = 0; i < n; ++i) {
    if (i == 0) gram_range(0, 0, mats[0].ntiles);
    if (i + 1 < n) {
      const int h = mats[i + 1].ntiles < head ? mats[i + 1].ntiles : head;
      gram_range(i + 1, 0, h);
      combine_all(i);
      gram_range(i + 1, h, mats[i + 1].ntiles);
    } else {
      combine_all(i);
    }
  }
  plan.n_items = static_cast<int>(items.size());
  if (plan.grid > plan.n_items) plan.grid = plan.n_items;
  if (cudaMalloc(&plan.d_items, sizeof(FusedItem) * items.size()) != cudaSuccess) {
    plan.d_items = nullptr;
    return NGALORE_ERR_ALLOC;
  }
  if (cudaMemcpy(plan.d_items, items.data(), sizeof(FusedItem) * items.size(), cudaMemcpyHostToDevice) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  return NGALORE_OK;
}

inline void fused_plan_destroy(FusedPlan& plan) {
  if (plan.d_items) cudaFree(plan.d_items);
  plan.d_items = nullptr;
}

inline ngalore_status fused_stream_launch(FusedPlan& plan, const MatDesc* d_mats, int /*n_mats*/, Ctrl* d_ctrl,
                                          const Hyper* d_hyper, int s, cudaStream_t stream, int64_t* launches) {
  if (s <= 8)
    fused_stream_kernel<8><<<plan.grid, kStreamThreads, 0, stream>>>(d_mats, plan.d_items, plan.n_items, d_ctrl, d_hyper, plan.tile_elems);
  else if (s <= 16)
    fused_stream_kernel<16><<<plan.grid, kStreamThreads, 0, stream>>>(d_mats, plan.d_items, plan.n_items, d_ctrl, d_hyper, plan.tile_elems);
  else
    fused_stream_kernel<32><<<plan.grid, kStreamThreads, 0, stream>>>(d_mats, plan.d_items, plan.n_items, d_ctrl, d_hyper, plan.tile_elems);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

}  // namespace ngalore
