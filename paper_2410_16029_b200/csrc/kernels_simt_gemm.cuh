// A plain strided SIMT GEMM.  It is the debug path of the two projection GEMMs and the workhorse
// of the small dense products of the subspace refresh (Gram matrices).
#pragma once

#include "common.cuh"

namespace ngalore {

enum SimtDtype { DT_BF16 = 0, DT_F32 = 1, DT_F64 = 2, DT_F16 = 3 };
enum SimtEpilogue {
  EPI_STORE = 0,      // C = acc
  EPI_W_UPDATE = 1,   // C = (1 - lr wd) C - lr acc          (Sec. 2.2 update; decoupled decay)
  EPI_ACCUMULATE = 2  // C += acc
};

struct SimtGemm {
  int m, n, k;
  const void* A;   // A(i, kk) at A[i * a_rs + kk * a_cs]
  const void* A2;  // optional second operand added to A on load (same strides and dtype)
  long long a_rs, a_cs;
  int a_dt;
  const void* B;   // B(kk, j) at B[kk * b_rs + j * b_cs]
  const void* B2;
  long long b_rs, b_cs;
  int b_dt;
  void* C;         // C(i, j) at C[i * c_rs + j * c_cs]
  long long c_rs, c_cs;
  int c_dt;
  int epilogue;
  const Hyper* hyper;    // EPI_W_UPDATE only
  const int* skip_flag;  // optional: when *skip_flag != 0 the kernel leaves C untouched
};

template <typename Acc>
__device__ __forceinline__ Acc simt_load(const void* p, int dt, long long idx) {
  if (dt == DT_BF16) return static_cast<Acc>(__bfloat162float(static_cast<const __nv_bfloat16*>(p)[idx]));
  if (dt == DT_F16) return static_cast<Acc>(__half2float(static_cast<const __half*>(p)[idx]));
  if (dt == DT_F32) return static_cast<Acc>(static_cast<const float*>(p)[idx]);
  return static_cast<Acc>(static_cast<const double*>(p)[idx]);
}

template <typename Acc>
__global__ void __launch_bounds__(256) simt_gemm_kernel(SimtGemm g) {
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ Acc As[BK][BM + 1];
  __shared__ Acc Bs[BK][BN + 1];
  if (g.skip_flag != nullptr && *g.skip_flag != 0) return;
  const int t = threadIdx.x;
  const int tx = t & 15, ty = t >> 4;
  const int i0 = blockIdx.y * BM, j0 = blockIdx.x * BN;
  Acc acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = Acc(0);

  const bool a_k_contig = (g.a_cs == 1);
  const bool b_n_contig = (g.b_cs == 1);
  for (int k0 = 0; k0 < g.k; k0 += BK) {
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      int i, kk;
      if (a_k_contig) { kk = t & 15; i = (t >> 4) + 16 * p; } else { i = t & 63; kk = (t >> 6) + 4 * p; }
      Acc val = Acc(0);
      if (i0 + i < g.m && k0 + kk < g.k) {
        const long long idx = static_cast<long long>(i0 + i) * g.a_rs + static_cast<long long>(k0 + kk) * g.a_cs;
        val = simt_load<Acc>(g.A, g.a_dt, idx);
        if (g.A2 != nullptr) val += simt_load<Acc>(g.A2, g.a_dt, idx);
      }
      As[kk][i] = val;
      int j, kb;
      if (b_n_contig) { j = t & 63; kb = (t >> 6) + 4 * p; } else { kb = t & 15; j = (t >> 4) + 16 * p; }
      Acc vb = Acc(0);
      if (j0 + j < g.n && k0 + kb < g.k) {
        const long long idx = static_cast<long long>(k0 + kb) * g.b_rs + static_cast<long long>(j0 + j) * g.b_cs;
        vb = simt_load<Acc>(g.B, g.b_dt, idx);
        if (g.B2 != nullptr) vb += simt_load<Acc>(g.B2, g.b_dt, idx);
      }
      Bs[kb][j] = vb;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      Acc a[4], b[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) { a[x] = As[kk][ty * 4 + x]; b[x] = Bs[kk][tx * 4 + x]; }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] += a[x] * b[y];
    }
    __syncthreads();
  }

  float lr = 0.f, decay = 1.f;
  if (g.epilogue == EPI_W_UPDATE) { lr = g.hyper->lr; decay = 1.f - g.hyper->lr * g.hyper->wd; }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = i0 + ty * 4 + x;
    if (i >= g.m) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int j = j0 + tx * 4 + y;
      if (j >= g.n) continue;
      const long long idx = static_cast<long long>(i) * g.c_rs + static_cast<long long>(j) * g.c_cs;
      Acc val = acc[x][y];
      if (g.epilogue == EPI_W_UPDATE) {
        float* c = static_cast<float*>(g.C);
        c[idx] = decay * c[idx] - lr * static_cast<float>(val);
        continue;
      }
      if (g.epilogue == EPI_ACCUMULATE) val += simt_load<Acc>(g.C, g.c_dt, idx);
      if (g.c_dt == DT_F32) static_cast<float*>(g.C)[idx] = static_cast<float>(val);
      else if (g.c_dt == DT_F64) static_cast<double*>(g.C)[idx] = static_cast<double>(val);
      else static_cast<__nv_bfloat16*>(g.C)[idx] = __float2bfloat16_rn(static_cast<float>(val));
    }
  }
}

template <typename Acc>
inline cudaError_t launch_simt_gemm(const SimtGemm& g, cudaStream_t stream) {
  if (g.m <= 0 || g.n <= 0) return cudaSuccess;
  dim3 grid((g.n + 63) / 64, (g.m + 63) / 64);
  simt_gemm_kernel<Acc><<<grid, 256, 0, stream>>>(g);
  return cudaGetLastError();
}

}  // namespace ngalore
