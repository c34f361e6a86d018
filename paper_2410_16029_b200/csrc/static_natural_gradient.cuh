// ngalore_natural_gradient_static: the natural-gradient transform of one matrix for callers that
// must not allocate device memory.  The per-tile Gram partials and the solved weights, which the
// optimizer state normally keeps in memory obtained from cudaMalloc, live here in a fixed array
// that is part of the library image.  Include this file from exactly one .cu file: the array, the
// kernels that use it and the host code that asks the runtime for its device address must be in
// the same translation unit.
#pragma once

#include <atomic>

#include "../../include/ngalore.h"
#include "common.cuh"
#include "kernels_stream.cuh"

namespace ngalore {

constexpr int kStaticTileElems = 8192;
constexpr int kStaticMaxTiles = 1024;  // => at most 8,388,608 elements per history slot
constexpr size_t kStaticPartBytes = static_cast<size_t>(kStaticMaxTiles) * kMaxHistory * sizeof(double);  // 256 KiB
constexpr size_t kStaticScratchBytes = kStaticPartBytes + 512;

// Layout: [0, kStaticPartBytes) per-tile partial Gram rows (tile-major, s doubles per tile);
// then kMaxHistory floats of weights; then two ints (skip flag, status when the caller passes none).
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticArgs {
  const float* H;
  long long n;
  int s, count, cur, ntiles;
  double lambda;
  double* K;
  float* out;
  int* status;
  unsigned char* scratch;  // device address of g_static_scratch
};

__device__ __forceinline__ MatDesc static_desc(const StaticArgs& a) {
  MatDesc d{};
  d.s = a.s;
  d.rn = a.n;
  d.H = const_cast<float*>(a.H);
  d.Kraw = a.K;
  d.gpart = reinterpret_cast<double*>(a.scratch);
  d.wsol = reinterpret_cast<float*>(a.scratch + kStaticPartBytes);
  d.step_bad = reinterpret_cast<int*>(a.scratch + kStaticPartBytes + kMaxHistory * sizeof(float));
  d.status = a.status != nullptr ? a.status : d.step_bad + 1;
  d.ntiles = a.ntiles;
  return d;
}

template <int SMAX>
__global__ void __launch_bounds__(kStreamThreads) static_gram_kernel(StaticArgs a) {
  __shared__ double red[(kStreamThreads / 32) * SMAX];
  const MatDesc d = static_desc(a);
  gram_tile<SMAX>(d, blockIdx.x, a.cur, a.count, kStaticTileElems, red);
}

__global__ void __launch_bounds__(32) static_solve_kernel(StaticArgs a) {
  __shared__ double A[kMaxHistory * (kMaxHistory + 1)];
  const MatDesc d = static_desc(a);
  solve_matrix(d, a.cur, a.count, a.lambda, A);
}

// out = sum_j w_j H_j (zeros when the solve flagged the step).
template <int SMAX>
__global__ void __launch_bounds__(kStreamThreads) static_combine_kernel(StaticArgs a) {
  const MatDesc d = static_desc(a);
  const bool bad = *d.step_bad != 0;
  float w[SMAX];
#pragma unroll
  for (int j = 0; j < SMAX; ++j) w[j] = (j < a.count && !bad) ? d.wsol[j] : 0.f;
  const long long e0 = static_cast<long long>(blockIdx.x) * kStaticTileElems;
  const long long e1 = (e0 + kStaticTileElems < a.n) ? e0 + kStaticTileElems : a.n;
  for (long long e = e0 + threadIdx.x * 4; e < e1; e += kStreamThreads * 4) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < SMAX; ++j) {
      if (j < a.count) {
        const float4 y = ldg4(a.H + static_cast<long long>(j) * a.n + e);
        acc.x = fmaf(w[j], y.x, acc.x);
        acc.y = fmaf(w[j], y.y, acc.y);
        acc.z = fmaf(w[j], y.z, acc.z);
        acc.w = fmaf(w[j], y.w, acc.w);
      }
    }
    *reinterpret_cast<float4*>(a.out + e) = acc;
  }
}

// Device address of the scratch array, looked up once per device (the array's name is only a
// host-side handle in host code; kernels must be given the address the runtime reports).
inline cudaError_t static_scratch_address(unsigned char** out) {
  constexpr int kMaxDevices = 64;
  static std::atomic<unsigned char*> cached[kMaxDevices];  // zero-initialised; threads may race to fill an entry
  int dev = 0;                                             // with the same value
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  unsigned char* addr = cached[dev].load(std::memory_order_acquire);
  if (addr == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    addr = static_cast<unsigned char*>(p);
    cached[dev].store(addr, std::memory_order_release);
  }
  *out = addr;
  return cudaSuccess;
}

template <int SMAX>
inline cudaError_t static_launch(const StaticArgs& a, cudaStream_t stream) {
  static_gram_kernel<SMAX><<<a.ntiles, kStreamThreads, 0, stream>>>(a);
  static_solve_kernel<<<1, 32, 0, stream>>>(a);
  static_combine_kernel<SMAX><<<a.ntiles, kStreamThreads, 0, stream>>>(a);
  return cudaGetLastError();
}

}  // namespace ngalore

extern "C" ngalore_status ngalore_natural_gradient_static(const float* H, int64_t n, int s, int count, int cur,
                                                          double lambda, double* K, float* out, int* status,
                                                          void* stream) {
  using namespace ngalore;
  if (H == nullptr || K == nullptr || out == nullptr) return NGALORE_ERR_INVALID_ARG;
  if (s < 1 || s > kMaxHistory || count < 1 || count > s || cur < 0 || cur >= count) return NGALORE_ERR_INVALID_ARG;
  if (n < 4 || n % 4 != 0 || !(lambda > 0.0)) return NGALORE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(H) | reinterpret_cast<uintptr_t>(out)) & 15u) return NGALORE_ERR_INVALID_ARG;
  const long long ntiles = (n + kStaticTileElems - 1) / kStaticTileElems;
  if (ntiles > kStaticMaxTiles) return NGALORE_ERR_INVALID_ARG;  // beyond the fixed scratch: n > 8,388,608
  StaticArgs a{};
  if (static_scratch_address(&a.scratch) != cudaSuccess) return NGALORE_ERR_CUDA;
  a.H = H; a.n = n; a.s = s; a.count = count; a.cur = cur; a.ntiles = static_cast<int>(ntiles);
  a.lambda = lambda; a.K = K; a.out = out; a.status = status;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = s <= 8 ? static_launch<8>(a, st) : (s <= 16 ? static_launch<16>(a, st) : static_launch<32>(a, st));
  return e == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}
