// Streaming kernels of the step: Gram row of the history ring, the s x s Cholesky solve,
// and the fused natural-gradient combination + Adam moments (Sec. 2.4 and Sec. 2.2).
#pragma once

#include "common.cuh"

namespace ngalore {

__device__ __forceinline__ float4 ldg4(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// Partial inner products <H_cur, H_j> over one tile of the flattened r' x N index range.
// Products and short per-thread sums are fp32; everything across threads is fp64.
template <int SMAX>
__device__ __forceinline__ void gram_tile(const MatDesc& d, int local, int cur, int c, int tile_elems,
                                          double* red /* smem: (kStreamThreads/32) * SMAX */) {
  const long long e0 = static_cast<long long>(local) * tile_elems;
  const long long e1 = (e0 + tile_elems < d.rn) ? e0 + tile_elems : d.rn;
  float acc[SMAX];
#pragma unroll
  for (int j = 0; j < SMAX; ++j) acc[j] = 0.f;
  const float* Hc = d.H + static_cast<long long>(cur) * d.rn;
  for (long long e = e0 + threadIdx.x * 4; e < e1; e += kStreamThreads * 4) {
    const float4 x = ldg4(Hc + e);
#pragma unroll
    for (int j = 0; j < SMAX; ++j) {
      if (j < c) {
        const float4 y = ldg4(d.H + static_cast<long long>(j) * d.rn + e);
        acc[j] += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
      }
    }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int j = 0; j < SMAX; ++j) {
    const double t = warp_sum(static_cast<double>(acc[j]));
    if (lane == 0) red[warp * SMAX + j] = t;
  }
  __syncthreads();
  if (threadIdx.x < SMAX) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kStreamThreads / 32; ++w) t += red[w * SMAX + threadIdx.x];
    if (static_cast<int>(threadIdx.x) < d.s) {
      d.gpart[static_cast<long long>(local) * d.s + threadIdx.x] = t;
      __threadfence();  // a later reader may run in another CTA of the same launch
    }
  }
  __syncthreads();
}

// One warp: finish the Gram row from the per-tile partials (fixed order, so the result is
// reproducible), form lambda I + K with K = Kraw / c, factor it (Cholesky, fp64) and solve for
// the weights w of N~ = sum_i w_i H_i, i.e. (lambda I + K) w = e_cur.  This is F^-1 applied to the
// current gradient by the Woodbury identity, written for the case where the current gradient is a
// column of the stacked matrix; it avoids the cancellation of the two-term form.
// A is warp-private shared memory of kMaxHistory x (kMaxHistory + 1) doubles.
// presum (optional, shared memory): groups x stride partial sums of the Gram row, already reduced over
// disjoint subsets of the tiles by the caller.
__device__ __forceinline__ void solve_matrix(const MatDesc& d, int cur, int c, double lambda, double* A,
                                             const double* presum = nullptr, int groups = 0, int stride = 0) {
  const int lane = threadIdx.x & 31;
  constexpr int LD = kMaxHistory + 1;
  bool finite = true;
  // Gram row: lane j sums tile partials of column j.
  if (d.s > 0) {
    double row = 0.0;
    if (lane < c) {
      if (presum != nullptr) {
        for (int g = 0; g < groups; ++g) row += presum[g * stride + lane];
      } else {
        for (int t = 0; t < d.ntiles; ++t) row += __ldcg(d.gpart + static_cast<long long>(t) * d.s + lane);
      }
      if (!isfinite(row)) finite = false;
    }
    finite = __all_sync(0xffffffffu, finite);
    if (lane < c) {
      const double val = finite ? row : 0.0;
      d.Kraw[cur * d.s + lane] = val;
      d.Kraw[lane * d.s + cur] = val;
    }
    __syncwarp();
  }
  int bad = finite ? 0 : 7 /* NGALORE_ERR_NONFINITE */;
  // A = lambda I + Kraw / c on the c valid slots.
  for (int i = 0; i < c; ++i) {
    if (lane < c) {
      double a = d.s > 0 ? d.Kraw[i * d.s + lane] / static_cast<double>(c) : 0.0;
      if (i == lane) a += lambda;
      A[i * LD + lane] = a;
    }
  }
  __syncwarp();
  // Cholesky, lower factor stored in place; lane = row.
  for (int k = 0; k < c && bad == 0; ++k) {
    const double dkk = A[k * LD + k];
    if (!(dkk > 0.0) || !isfinite(dkk)) {
      bad = isfinite(dkk) ? 6 /* NGALORE_ERR_NOT_SPD */ : 7;
      break;
    }
    const double lkk = sqrt(dkk);
    __syncwarp();
    if (lane == k) A[k * LD + k] = lkk;
    if (lane > k && lane < c) A[lane * LD + k] /= lkk;
    __syncwarp();
    if (lane > k && lane < c) {
      const double lik = A[lane * LD + k];
      for (int j = k + 1; j <= lane; ++j) A[lane * LD + j] -= lik * A[j * LD + k];
    }
    __syncwarp();
  }
  // Forward and backward substitution (serial; c <= 32).
  if (lane == 0) {
    if (bad == 0) {
      double t[kMaxHistory], w[kMaxHistory];
      for (int i = 0; i < c; ++i) {
        double acc = (i == cur) ? 1.0 : 0.0;
        for (int j = 0; j < i; ++j) acc -= A[i * LD + j] * t[j];
        t[i] = acc / A[i * LD + i];
      }
      for (int i = c - 1; i >= 0; --i) {
        double acc = t[i];
        for (int j = i + 1; j < c; ++j) acc -= A[j * LD + i] * w[j];
        w[i] = acc / A[i * LD + i];
      }
      for (int i = 0; i < kMaxHistory; ++i) d.wsol[i] = i < c ? static_cast<float>(w[i]) : 0.f;
      *d.step_bad = 0;
    } else {
      for (int i = 0; i < kMaxHistory; ++i) d.wsol[i] = 0.f;
      *d.step_bad = 1;
      atomicCAS(d.status, 0, bad);
      // The poisoned slot becomes a zero gradient: its Gram row and column vanish.
      for (int j = 0; j < d.s; ++j) {
        d.Kraw[cur * d.s + j] = 0.0;
        d.Kraw[j * d.s + cur] = 0.0;
      }
    }
  }
  __syncwarp();
}


// N~ = sum_j w_j H_j, then the Adam moments as printed in Sec. 2.2 (eps inside the root, no bias
// correction), then u rounded to fp16 for the back-projection GEMM.
template <int SMAX>
__device__ __forceinline__ void combine_tile(const MatDesc& d, int local, int cur, int c, int tile_elems,
                                             const Hyper& hp, const float* wsm /* smem weights */) {
  const long long e0 = static_cast<long long>(local) * tile_elems;
  const long long e1 = (e0 + tile_elems < d.rn) ? e0 + tile_elems : d.rn;
  if (__ldcg(d.step_bad)) {
    float* Hc = d.H + static_cast<long long>(cur) * d.rn;
    for (long long e = e0 + threadIdx.x * 4; e < e1; e += kStreamThreads * 4) {
      *reinterpret_cast<float4*>(Hc + e) = make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<uint2*>(d.u16 + e) = make_uint2(0u, 0u);
    }
    return;
  }
  float w[SMAX];
#pragma unroll
  for (int j = 0; j < SMAX; ++j) w[j] = wsm[j];
  const float b1 = hp.beta1, b2 = hp.beta2, eps = hp.eps;
  for (long long e = e0 + threadIdx.x * 4; e < e1; e += kStreamThreads * 4) {
    float4 n = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < SMAX; ++j) {
      if (j < c) {
        const float4 y = ldg4(d.H + static_cast<long long>(j) * d.rn + e);
        n.x = fmaf(w[j], y.x, n.x);
        n.y = fmaf(w[j], y.y, n.y);
        n.z = fmaf(w[j], y.z, n.z);
        n.w = fmaf(w[j], y.w, n.w);
      }
    }
    float4 m = ldg4(d.m + e), v = ldg4(d.v + e);
    m.x = b1 * m.x + (1.f - b1) * n.x;
    m.y = b1 * m.y + (1.f - b1) * n.y;
    m.z = b1 * m.z + (1.f - b1) * n.z;
    m.w = b1 * m.w + (1.f - b1) * n.w;
    v.x = b2 * v.x + (1.f - b2) * n.x * n.x;
    v.y = b2 * v.y + (1.f - b2) * n.y * n.y;
    v.z = b2 * v.z + (1.f - b2) * n.z * n.z;
    v.w = b2 * v.w + (1.f - b2) * n.w * n.w;
    *reinterpret_cast<float4*>(d.m + e) = m;
    *reinterpret_cast<float4*>(d.v + e) = v;
    const float u0 = m.x / sqrtf(v.x + eps), u1 = m.y / sqrtf(v.y + eps);
    const float u2 = m.z / sqrtf(v.z + eps), u3 = m.w / sqrtf(v.w + eps);
    *reinterpret_cast<uint2*>(d.u16 + e) = pack_f16x4(u0, u1, u2, u3);
  }
}

// ---------------------------------------------------------------- plain (debug) kernels: one launch per phase

template <int SMAX>
__global__ void __launch_bounds__(kStreamThreads) gram_kernel(const MatDesc* mats, const StreamTile* tiles,
                                                              const Ctrl* ctrl) {
  __shared__ double red[(kStreamThreads / 32) * SMAX];
  const StreamTile t = tiles[blockIdx.x];
  const MatDesc& d = mats[t.mat];
  if (d.s == 0) return;
  gram_tile<SMAX>(d, t.local, ring_cur(ctrl, d.s), ring_count(ctrl, d.s), d.te, red);
}

__global__ void __launch_bounds__(128) solve_kernel(const MatDesc* mats, int n_mats, const Ctrl* ctrl,
                                                    const Hyper* hyper) {
  __shared__ double A[4][kMaxHistory * (kMaxHistory + 1)];
  const int warp = threadIdx.x >> 5;
  const int mat = blockIdx.x * 4 + warp;
  if (mat >= n_mats) return;
  const MatDesc& d = mats[mat];
  if (d.s == 0) return;
  solve_matrix(d, ring_cur(ctrl, d.s), ring_count(ctrl, d.s), hyper->lambda, A[warp]);
}

template <int SMAX>
__global__ void __launch_bounds__(kStreamThreads) combine_kernel(const MatDesc* mats, const StreamTile* tiles,
                                                                 const Ctrl* ctrl, const Hyper* hyper) {
  __shared__ float wsm[kMaxHistory];
  const StreamTile t = tiles[blockIdx.x];
  const MatDesc& d = mats[t.mat];
  if (threadIdx.x < kMaxHistory) wsm[threadIdx.x] = d.wsol[threadIdx.x];
  __syncthreads();
  combine_tile<SMAX>(d, t.local, ring_cur(ctrl, d.s), ring_count(ctrl, d.s), d.te, *hyper, wsm);
}

__global__ void advance_kernel(Ctrl* ctrl) {
  ctrl->n_appended += 1;
  ctrl->k += 1;
  ctrl->epoch += 1;
  ctrl->work_counter = 0u;
  ctrl->gemm_counter0 = 0u;
  ctrl->gemm_counter1 = 0u;
  ctrl->spin_limit = 0;
  ctrl->debug_withhold = 0;
}

}  // namespace ngalore
