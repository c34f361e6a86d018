// The step for small ranks (r' <= 8: the fine-tuning regime of Sec. 4.2 and 4.3, ranks 4 and 8) as two bandwidth
// kernels without tensor cores.  At these ranks the low-rank state is a sliver (8 x N against M x N), the GEMMs
// are 8 multiply-adds per element of G or W, and the step is the traffic of G (2 bytes per element, once) and of
// W (4 bytes read, 4 written): so every element of G and W is touched exactly once, by plain loads and stores, and
// everything in between rides along:
//
//   sr_project_gram_kernel   one CTA per strip of 64 columns of one matrix: R strip = P^T G[:, strip] over all M rows
//                            (Sec. 1 projection), written into ring slot `cur` (Sec. 2.4), and the strip's share of
//                            the new Gram row <R, H_j> (Sec. 2.2 / 2.4) as a partial row in fp64.
//   sr_update_kernel         one CTA per strip again: add the partial rows of the matrix in a fixed order, solve
//                            (lambda I + K / c) w = e_cur by Cholesky in fp64 (Sec. 2.4; every CTA of a matrix
//                            solves the s x s system for itself, the CTA of strip 0 records the Gram row, the
//                            weights and the status), N~ strip = sum_j w_j H_j strip, the Adam moments (Sec. 2.2),
//                            u strip, and W[:, strip] <- (1 - lr wd) W - lr P u over all M rows (Sec. 2.2 update).
//
// Strips are handed out from a list ordered by falling M through a counter, so the long strips of a tall matrix
// (an embedding) start first.  Both kernels use the bf16-rounded projector the tensor-core path uses (Pt16 in the
// first, P16 in the second: the same values), so the two paths agree to rounding.
#pragma once

#include <algorithm>
#include <vector>

#include "../../include/ngalore.h"
#include "common.cuh"
#include "kernels_stream.cuh"

namespace ngalore {

constexpr int kSrRank = 8;        // rows of the low-rank matrices, padded with zero rows of P below
constexpr int kSrStrip = 64;      // columns per strip
constexpr int kSrThreads = 256;
constexpr int kSrPChunk = 512;    // rows of P staged in shared memory at a time
constexpr int kSrSMax = 16;       // longest history this path takes

struct SrItem {
  int mat;
  int n0;      // first column of the strip
  int strip;   // index of the strip within its matrix
  int pad;
};

struct SrMat {
  double* part;   // n_strips x s partial Gram rows
  int n_strips;
  int pad;
};

struct SrPlan {
  bool ready = false;
  SrItem* d_items = nullptr;
  SrMat* d_mats = nullptr;
  double* d_part = nullptr;
  int n_items = 0;
  int grid = 0;
  size_t device_bytes = 0;
};

__device__ __forceinline__ float sr_bf16_to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// ------------------------------------------------------------------------------------------ projection + Gram row

template <int SMAX>
__global__ void __launch_bounds__(kSrThreads) sr_project_gram_kernel(const MatDesc* __restrict__ mats, const SrMat* __restrict__ srm,
                                                                    const SrItem* __restrict__ items, int n_items,
                                                                    const uint16_t* const* __restrict__ Gptr, Ctrl* ctrl) {
  __shared__ float Ps[kSrRank][kSrPChunk];              // P^T, a chunk of rows at a time (16 KB)
  __shared__ float Rs[kSrThreads / 32][kSrRank][kSrStrip];  // per-warp partial R strips
  __shared__ double red[kSrThreads / 32][SMAX];
  __shared__ int s_item;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ct = tid & 7;          // column thread: columns 8 ct .. 8 ct + 7 of the strip
  const int rg = tid >> 3;         // row group 0 .. 31
  while (true) {
    if (tid == 0) s_item = static_cast<int>(atomicAdd(&ctrl->gemm_counter0, 1u));
    __syncthreads();
    const int it = s_item;
    if (it >= n_items) break;
    const SrItem item = items[it];
    const MatDesc& d = mats[item.mat];
    const int M = d.M, N = d.N, rp = d.rp;
    const uint16_t* __restrict__ G = Gptr[item.mat];
    const int col0 = item.n0 + 8 * ct;
    const bool col_ok = col0 < N;                       // N is a multiple of 8: a thread's eight columns are in or out
    float acc[kSrRank][8];
#pragma unroll
    for (int k = 0; k < kSrRank; ++k)
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[k][c] = 0.f;
    for (int m0 = 0; m0 < M; m0 += kSrPChunk) {
      const int rows = min(kSrPChunk, M - m0);
      __syncthreads();                                  // the previous chunk of P is no longer read
      for (int x = tid; x < kSrRank * kSrPChunk; x += kSrThreads) {
        const int k = x / kSrPChunk, m = x - k * kSrPChunk;
        Ps[k][m] = (k < rp && m < rows) ? sr_bf16_to_float(d.Pt16[static_cast<long long>(k) * d.ldpt + m0 + m]) : 0.f;
      }
      __syncthreads();
      if (col_ok) {
#pragma unroll 4
        for (int m = rg; m < rows; m += kSrThreads / 8) {
          const uint4 g = *reinterpret_cast<const uint4*>(G + static_cast<long long>(m0 + m) * N + col0);
          float gv[8];
          gv[0] = __uint_as_float(g.x << 16); gv[1] = __uint_as_float(g.x & 0xFFFF0000u);
          gv[2] = __uint_as_float(g.y << 16); gv[3] = __uint_as_float(g.y & 0xFFFF0000u);
          gv[4] = __uint_as_float(g.z << 16); gv[5] = __uint_as_float(g.z & 0xFFFF0000u);
          gv[6] = __uint_as_float(g.w << 16); gv[7] = __uint_as_float(g.w & 0xFFFF0000u);
#pragma unroll
          for (int k = 0; k < kSrRank; ++k) {
            const float p = Ps[k][m];
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[k][c] = fmaf(p, gv[c], acc[k][c]);
          }
        }
      }
    }
    // the four row groups of a warp by shuffles, then the eight warps through shared memory
#pragma unroll
    for (int k = 0; k < kSrRank; ++k)
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        float v = acc[k][c];
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        if (lane < 8) Rs[warp][k][8 * lane + c] = v;
      }
    __syncthreads();
    const int cur = ring_cur(ctrl, d.s), cnt = ring_count(ctrl, d.s);
    float* Hcur = current_gradient(d, cur);
    // the strip: element e = k * 64 + n for this thread's two elements; stored into slot `cur`
    float rv[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int e = tid + q * kSrThreads, k = e >> 6, n = e & 63;
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < kSrThreads / 32; ++w) v += Rs[w][k][n];
      rv[q] = v;
      if (k < rp && item.n0 + n < N) Hcur[static_cast<long long>(k) * N + item.n0 + n] = v;
    }
    // the strip's share of the Gram row: the entry of `cur` goes through the same operations as the others
    if (d.s > 0) {
#pragma unroll
      for (int j = 0; j < SMAX; ++j) {
        if (j < cnt) {
          float t = 0.f;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int e = tid + q * kSrThreads, k = e >> 6, n = e & 63;
            if (k < rp && item.n0 + n < N) {
              const float h = (j == cur) ? rv[q] : d.H[static_cast<long long>(j) * d.rn + static_cast<long long>(k) * N + item.n0 + n];
              t += rv[q] * h;
            }
          }
          const double s = warp_sum(static_cast<double>(t));
          if (lane == 0) red[warp][j] = s;
        }
      }
      __syncthreads();
      if (tid < cnt) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < kSrThreads / 32; ++w) t += red[w][tid];
        srm[item.mat].part[static_cast<long long>(item.strip) * d.s + tid] = t;
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------ solve + moments + W update

template <int SMAX>
__global__ void __launch_bounds__(kSrThreads) sr_update_kernel(const MatDesc* __restrict__ mats, const SrMat* __restrict__ srm,
                                                              const SrItem* __restrict__ items, int n_items,
                                                              float* const* __restrict__ Wptr, Ctrl* ctrl,
                                                              const Hyper* __restrict__ hyper) {
  __shared__ double A[kMaxHistory * (kMaxHistory + 1)];
  __shared__ double row[SMAX];
  __shared__ float wsm[SMAX];
  __shared__ float us[kSrRank][kSrStrip];
  __shared__ int s_item, s_bad;
  const int tid = threadIdx.x, lane = tid & 31;
  const Hyper hp = *hyper;
  constexpr int LD = kMaxHistory + 1;
  while (true) {
    if (tid == 0) s_item = static_cast<int>(atomicAdd(&ctrl->gemm_counter1, 1u));
    __syncthreads();
    const int it = s_item;
    if (it >= n_items) break;
    const SrItem item = items[it];
    const MatDesc& d = mats[item.mat];
    const int M = d.M, N = d.N, rp = d.rp;
    const int cur = ring_cur(ctrl, d.s), cnt = ring_count(ctrl, d.s);
    const bool writer = item.strip == 0;      // this CTA records the Gram row, the weights and the status
    // ---- Gram row (fixed order over the strips), system matrix, Cholesky solve: one warp
    if (tid < 32) {
      int bad = 0;
      if (d.s > 0) {
        double r = 0.0;
        if (lane < cnt) {
          const SrMat sm = srm[item.mat];
          for (int t = 0; t < sm.n_strips; ++t) r += sm.part[static_cast<long long>(t) * d.s + lane];
        }
        const bool finite = __all_sync(0xffffffffu, lane >= cnt || isfinite(r));
        if (!finite) bad = 7;                 // NGALORE_ERR_NONFINITE
        if (lane < cnt) row[lane] = finite ? r : 0.0;
        __syncwarp();
        // A = lambda I + K / c with K's row and column `cur` from this step, the rest as kept
        for (int i = 0; i < cnt; ++i)
          if (lane < cnt) {
            const double kij = (i == cur) ? row[lane] : (lane == cur ? row[i] : d.Kraw[i * d.s + lane]);
            A[i * LD + lane] = kij / static_cast<double>(cnt) + (i == lane ? hp.lambda : 0.0);
          }
        __syncwarp();
        for (int k = 0; k < cnt && bad == 0; ++k) {
          const double dkk = A[k * LD + k];
          if (!(dkk > 0.0) || !isfinite(dkk)) { bad = isfinite(dkk) ? 6 : 7; break; }
          const double lkk = sqrt(dkk);
          __syncwarp();
          if (lane == k) A[k * LD + k] = lkk;
          if (lane > k && lane < cnt) A[lane * LD + k] /= lkk;
          __syncwarp();
          if (lane > k && lane < cnt) {
            const double lik = A[lane * LD + k];
            for (int j = k + 1; j <= lane; ++j) A[lane * LD + j] -= lik * A[j * LD + k];
          }
          __syncwarp();
        }
        if (lane == 0) {
          double t[kMaxHistory], w[kMaxHistory];
          if (bad == 0) {
            for (int i = 0; i < cnt; ++i) {
              double a = (i == cur) ? 1.0 : 0.0;
              for (int j = 0; j < i; ++j) a -= A[i * LD + j] * t[j];
              t[i] = a / A[i * LD + i];
            }
            for (int i = cnt - 1; i >= 0; --i) {
              double a = t[i];
              for (int j = i + 1; j < cnt; ++j) a -= A[j * LD + i] * w[j];
              w[i] = a / A[i * LD + i];
            }
          }
          for (int i = 0; i < SMAX; ++i) wsm[i] = (bad == 0 && i < cnt) ? static_cast<float>(w[i]) : 0.f;
          s_bad = bad;
          if (writer) {
            for (int j = 0; j < d.s; ++j) {
              const double v = (bad == 0 && j < cnt) ? row[j] : 0.0;   // a poisoned slot becomes a zero gradient
              if (j < cnt || bad != 0) { d.Kraw[cur * d.s + j] = v; d.Kraw[j * d.s + cur] = v; }
            }
            for (int i = 0; i < kMaxHistory; ++i) d.wsol[i] = i < SMAX ? wsm[i] : 0.f;
            *d.step_bad = bad != 0 ? 1 : 0;
            if (bad != 0) atomicCAS(d.status, 0, bad);
          }
        }
      } else if (lane == 0) {
        wsm[0] = 1.f;                          // s = 0: the natural gradient is the projected gradient itself
        s_bad = 0;
        if (writer) *d.step_bad = 0;
      }
    }
    __syncthreads();
    const bool bad = s_bad != 0;
    // ---- natural gradient, moments and direction of the strip (two elements per thread)
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int e = tid + q * kSrThreads, k = e >> 6, n = e & 63;
      float u = 0.f;
      if (k < rp && item.n0 + n < N) {
        const long long off = static_cast<long long>(k) * N + item.n0 + n;
        if (bad) {
          current_gradient(d, cur)[off] = 0.f;
        } else {
          float nat = 0.f;
          if (d.s > 0) {
#pragma unroll
            for (int j = 0; j < SMAX; ++j)
              if (j < cnt) nat = fmaf(wsm[j], d.H[static_cast<long long>(j) * d.rn + off], nat);
          } else {
            nat = d.H[off];
          }
          const float mm = hp.beta1 * d.m[off] + (1.f - hp.beta1) * nat;
          const float vv = hp.beta2 * d.v[off] + (1.f - hp.beta2) * nat * nat;
          d.m[off] = mm;
          d.v[off] = vv;
          u = mm / sqrtf(vv + hp.eps);
        }
      }
      us[k][n] = u;
    }
    __syncthreads();
    // ---- W[:, strip] <- (1 - lr wd) W - lr P u: 16 column threads of four columns, 16 row groups
    if (!bad) {
      const int ct = tid & 15, rg = tid >> 4;
      const int col = item.n0 + 4 * ct;
      if (col < N) {
        float ur[kSrRank][4];
#pragma unroll
        for (int k = 0; k < kSrRank; ++k)
#pragma unroll
          for (int c = 0; c < 4; ++c) ur[k][c] = us[k][4 * ct + c];
        float* __restrict__ W = Wptr[item.mat];
        const float decay = 1.f - hp.lr * hp.wd;
        const __half* P16 = reinterpret_cast<const __half*>(d.P16);
#pragma unroll 4
        for (int m = rg; m < M; m += kSrThreads / 16) {
          const uint4 pb = *reinterpret_cast<const uint4*>(P16 + static_cast<long long>(m) * d.ldp);   // ldp is a multiple of 8
          const __half2* ph = reinterpret_cast<const __half2*>(&pb);
          float p[8];
#pragma unroll
          for (int x = 0; x < 4; ++x) { const float2 f = __half22float2(ph[x]); p[2 * x] = f.x; p[2 * x + 1] = f.y; }
          float4 w = *reinterpret_cast<const float4*>(W + static_cast<long long>(m) * N + col);
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
          for (int k = 0; k < kSrRank; ++k) {
            a0 = fmaf(p[k], ur[k][0], a0); a1 = fmaf(p[k], ur[k][1], a1);
            a2 = fmaf(p[k], ur[k][2], a2); a3 = fmaf(p[k], ur[k][3], a3);
          }
          w.x = decay * w.x - hp.lr * a0; w.y = decay * w.y - hp.lr * a1;
          w.z = decay * w.z - hp.lr * a2; w.w = decay * w.w - hp.lr * a3;
          *reinterpret_cast<float4*>(W + static_cast<long long>(m) * N + col) = w;
        }
      }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------ host side

// Can this set of matrices take the small-rank path?  Every r' <= 8, left projection, fp32 history and moments,
// s <= 16, columns a multiple of 8 (always true), and P16's rows padded to 8 entries (ldp >= 8, always true).
inline bool sr_eligible(const std::vector<MatDesc>& mats, int s) {
  if (s > kSrSMax) return false;
  for (const MatDesc& d : mats)
    if (d.rp > kSrRank || d.right != 0 || d.H16 != nullptr || d.m16 != nullptr) return false;
  return !mats.empty();
}

inline void sr_plan_destroy(SrPlan& plan) {
  if (plan.d_items) cudaFree(plan.d_items);
  if (plan.d_mats) cudaFree(plan.d_mats);
  if (plan.d_part) cudaFree(plan.d_part);
  plan.d_items = nullptr; plan.d_mats = nullptr; plan.d_part = nullptr;
  plan.ready = false;
}

inline ngalore_status sr_plan_create(SrPlan& plan, const std::vector<MatDesc>& mats, int s, int sm_count) {
  const int n = static_cast<int>(mats.size());
  std::vector<SrItem> items;
  std::vector<SrMat> srm(n);
  std::vector<long long> part_off(n);
  long long parts = 0;
  const int slots = s > 0 ? s : 1;
  for (int i = 0; i < n; ++i) {
    const int strips = (mats[i].N + kSrStrip - 1) / kSrStrip;
    part_off[i] = parts;
    parts += static_cast<long long>(strips) * slots;
    srm[i].n_strips = strips;
    srm[i].pad = 0;
    for (int t = 0; t < strips; ++t) items.push_back(SrItem{i, t * kSrStrip, t, 0});
  }
  std::stable_sort(items.begin(), items.end(), [&](const SrItem& a, const SrItem& b) { return mats[a.mat].M > mats[b.mat].M; });
  plan.n_items = static_cast<int>(items.size());
  plan.grid = std::min(plan.n_items, 2 * sm_count);
  if (cudaMalloc(&plan.d_items, sizeof(SrItem) * items.size()) != cudaSuccess) { plan.d_items = nullptr; return NGALORE_ERR_ALLOC; }
  if (cudaMalloc(&plan.d_mats, sizeof(SrMat) * n) != cudaSuccess) { plan.d_mats = nullptr; return NGALORE_ERR_ALLOC; }
  if (cudaMalloc(&plan.d_part, sizeof(double) * parts) != cudaSuccess) { plan.d_part = nullptr; return NGALORE_ERR_ALLOC; }
  for (int i = 0; i < n; ++i) srm[i].part = plan.d_part + part_off[i];
  if (cudaMemcpy(plan.d_items, items.data(), sizeof(SrItem) * items.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_mats, srm.data(), sizeof(SrMat) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemset(plan.d_part, 0, sizeof(double) * parts) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  plan.device_bytes = sizeof(SrItem) * items.size() + sizeof(SrMat) * n + sizeof(double) * parts;
  plan.ready = true;
  return NGALORE_OK;
}

// d_G / d_W: device arrays of the matrices' gradient and weight pointers.
inline ngalore_status sr_project_gram(const SrPlan& plan, const MatDesc* d_mats, const uint16_t* const* d_G, Ctrl* d_ctrl, int s,
                                      cudaStream_t stream, int64_t* launches) {
  if (s <= 8)
    sr_project_gram_kernel<8><<<plan.grid, kSrThreads, 0, stream>>>(d_mats, plan.d_mats, plan.d_items, plan.n_items, d_G, d_ctrl);
  else
    sr_project_gram_kernel<16><<<plan.grid, kSrThreads, 0, stream>>>(d_mats, plan.d_mats, plan.d_items, plan.n_items, d_G, d_ctrl);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

inline ngalore_status sr_update(const SrPlan& plan, const MatDesc* d_mats, float* const* d_W, Ctrl* d_ctrl, const Hyper* d_hyper,
                                int s, cudaStream_t stream, int64_t* launches) {
  if (s <= 8)
    sr_update_kernel<8><<<plan.grid, kSrThreads, 0, stream>>>(d_mats, plan.d_mats, plan.d_items, plan.n_items, d_W, d_ctrl, d_hyper);
  else
    sr_update_kernel<16><<<plan.grid, kSrThreads, 0, stream>>>(d_mats, plan.d_mats, plan.d_items, plan.n_items, d_W, d_ctrl, d_hyper);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

}  // namespace ngalore
