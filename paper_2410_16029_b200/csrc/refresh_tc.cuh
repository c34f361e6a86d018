// Subspace refresh on the tensor cores (Sec. 1: P spans the leading left singular vectors of G).
//
// Randomized subspace iteration with L = r' columns: Y = G Omega, then q sweeps of
//   Z = G^T Q_Y,  Q_Z = orth(Z),  Y = G Q_Z,  Q_Y = orth(Y).
// Every product runs through the grouped tcgen05 GEMM with the iterate split into a high and a low
// bf16 part (16 mantissa bits).  Between products the iterate only has to stay well conditioned, so
// orth() is a *shifted* Cholesky QR: the Gram matrix Y^T Y comes from the tensor cores (three bf16
// products, fp32 accumulation), its columns are scaled to unit norm and a small multiple of the identity
// is added before the fp64 Cholesky factorisation so that the fp32 accumulation error cannot make it
// indefinite, and
// Q = Y R^-1 is again a tensor-core GEMM with R^-1 split in two bf16 parts.  The last basis is then
// orthonormalised exactly (Gram, Cholesky and triangular solve in fp64), rotated to the Ritz vectors of G inside
// the subspace (Z = G^T Q, eigenvectors V of Z^T Z by the Jacobi kernels of ritz_jacobi.cuh, P = Q V on the tensor
// cores, columns in falling order of their singular value) and orthonormalised once more.
#pragma once

#include <cstring>
#include <vector>

#include <algorithm>

#include "gemm_tcgen05.cuh"
#include "kernels_refresh.cuh"
#include "ritz_jacobi.cuh"

namespace ngalore {

// hi = bf16(x), lo = bf16(x - hi); rows x cols fp32 (dense) -> rows x ld bf16 (padding untouched: it is zero).
__global__ void split_hilo_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ hi,
                                  __nv_bfloat16* __restrict__ lo, long long n, int cols, int ld) {
  const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (i >= n) return;
  const float x = src[i];
  const __nv_bfloat16 h = __float2bfloat16_rn(x);
  const long long o = (i / cols) * ld + (i % cols);
  hi[o] = h;
  lo[o] = __float2bfloat16_rn(x - __bfloat162float(h));
}

struct SplitJob {
  const float* src;
  __nv_bfloat16 *hi, *lo;
  long long n;
  int cols, ld;
};

// All matrices in one launch: blockIdx.y selects the matrix, blockIdx.x strides over its elements, four at a
// time where the row length allows it (the kernel is a pure stream: 4 bytes in, 4 bytes out per element).
__global__ void split_hilo_grouped_kernel(const SplitJob* jobs) {
  const SplitJob jb = jobs[blockIdx.y];
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  const long long t0 = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if ((jb.cols & 3) == 0 && (jb.ld & 3) == 0) {
    const int quads_per_row = jb.cols >> 2;
    for (long long q = t0; q < (jb.n >> 2); q += stride) {
      const float4 x = reinterpret_cast<const float4*>(jb.src)[q];
      const long long row = q / quads_per_row;
      const long long o = row * jb.ld + ((q - row * quads_per_row) << 2);
      const __nv_bfloat162 h01 = __floats2bfloat162_rn(x.x, x.y), h23 = __floats2bfloat162_rn(x.z, x.w);
      const __nv_bfloat162 l01 = __floats2bfloat162_rn(x.x - __low2float(h01), x.y - __high2float(h01));
      const __nv_bfloat162 l23 = __floats2bfloat162_rn(x.z - __low2float(h23), x.w - __high2float(h23));
      uint2 hv, lv;
      hv.x = *reinterpret_cast<const uint32_t*>(&h01); hv.y = *reinterpret_cast<const uint32_t*>(&h23);
      lv.x = *reinterpret_cast<const uint32_t*>(&l01); lv.y = *reinterpret_cast<const uint32_t*>(&l23);
      *reinterpret_cast<uint2*>(jb.hi + o) = hv;
      *reinterpret_cast<uint2*>(jb.lo + o) = lv;
    }
    return;
  }
  for (long long i = t0; i < jb.n; i += stride) {
    const float x = jb.src[i];
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    const long long o = (i / jb.cols) * jb.ld + (i % jb.cols);
    jb.hi[o] = h;
    jb.lo[o] = __float2bfloat16_rn(x - __bfloat162float(h));
  }
}

// Clear a list of buffers in one launch (a memset per buffer costs more in launch overhead than in work when
// there are hundreds of small ones): blockIdx.y selects the buffer, blockIdx.x strides over its 16-byte words.
struct ZeroJob {
  float4* p;
  long long n16;
};

__global__ void zero_jobs_kernel(const ZeroJob* jobs) {
  const ZeroJob jb = jobs[blockIdx.y];
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < jb.n16;
       i += static_cast<long long>(gridDim.x) * blockDim.x)
    jb.p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

struct GramPrep {
  const float* C32;  // L x L Gram matrix from the tensor cores
  double* C64;       // L x L, lower triangle written: column-scaled, symmetrised Gram + shift I (as doubles, or
                     // as L x L floats at the same address: gram_prep_kernel<float>)
  double* D;         // L column norms d_i = sqrt(C_ii)
  int L;
};

// Shift added to the unit-diagonal Gram matrix.  Each entry carries a relative error of at most about
// 3 * 2^-18 from the two-part bf16 split (the dropped lo*lo product and the rounding of lo) plus the fp32
// accumulation error, so the error matrix has norm below 2^-16 L; with this shift the Cholesky factorisation
// cannot meet a negative pivot.  The price is that directions closer than sqrt(shift) are not pulled
// apart, which is harmless between products.
__host__ __device__ inline double gram_shift(int L) { return static_cast<double>(L) / 65536.0; }

// One CTA per matrix: C64 = D^-1 ((C32 + C32^T) / 2) D^-1 + shift I with D = diag(sqrt(C_ii)).
// Scaling the columns to unit norm first makes the shift act on every column alike, whatever its
// norm, so weak directions are still orthogonalised against each other and re-normalised.
// (blockIdx.y shares the entries of a matrix among several CTAs; each of them forms the column norms for itself)
template <typename T>
__global__ void __launch_bounds__(256) gram_prep_kernel(const GramPrep* probs, double shift_scale) {
  __shared__ double Ds[880];
  const GramPrep p = probs[blockIdx.x];
  for (int i = threadIdx.x; i < p.L; i += 256) {
    const double c = static_cast<double>(p.C32[static_cast<long long>(i) * p.L + i]);
    Ds[i] = sqrt(fmax(c, 1e-60));
    if (blockIdx.y == 0) p.D[i] = Ds[i];
  }
  __syncthreads();
  const long long total = static_cast<long long>(p.L) * p.L;
  for (long long x = blockIdx.y * 256 + threadIdx.x; x < total; x += 256ll * gridDim.y) {
    const int i = static_cast<int>(x / p.L), j = static_cast<int>(x % p.L);
    if (j > i) continue;
    double v = 0.5 * (static_cast<double>(p.C32[x]) + static_cast<double>(p.C32[static_cast<long long>(j) * p.L + i]));
    v /= Ds[i] * Ds[j];
    if (i == j) v = 1.0 + shift_scale * gram_shift(p.L);
    reinterpret_cast<T*>(p.C64)[x] = static_cast<T>(v);
  }
}

struct SyrkTile {
  int mat, ti, tj, k0;  // output tile (ti, tj <= ti) of 64 x 64, rows k0 .. k0 + kSyrkRows of Y
};
constexpr int kSyrkRows = 1024;

struct SyrkMat {
  const float* Y;  // rows x L fp32
  double* C;       // L x L fp64 accumulator (zeroed before the launch); lower tiles are written
  int rows, L;
};

// Exact Gram matrix C += Y^T Y in fp64 (products of fp32 values are exact in fp64), grouped over all
// matrices: one CTA per 64 x 64 lower tile and slab of rows, partial sums added with fp64 atomics.
__global__ void __launch_bounds__(256) syrk_f64_kernel(const SyrkMat* mats, const SyrkTile* tiles) {
  __shared__ float As[16][64 + 4];
  __shared__ float Bs[16][64 + 4];
  const SyrkTile t = tiles[blockIdx.x];
  const SyrkMat m = mats[t.mat];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int i0 = t.ti * 64, j0 = t.tj * 64;
  const int k1 = (t.k0 + kSyrkRows < m.rows) ? t.k0 + kSyrkRows : m.rows;
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
  // the next 16 rows are fetched into registers while the current ones are multiplied
  const int lc = threadIdx.x & 63, lk = threadIdx.x >> 6;
  float pa[4], pb[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int k = k0 + lk + 4 * p;
      pa[p] = (k < k1 && i0 + lc < m.L) ? m.Y[static_cast<long long>(k) * m.L + i0 + lc] : 0.f;
      pb[p] = (k < k1 && j0 + lc < m.L) ? m.Y[static_cast<long long>(k) * m.L + j0 + lc] : 0.f;
    }
  };
  fetch(t.k0);
  for (int k0 = t.k0; k0 < k1; k0 += 16) {
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      As[lk + 4 * p][lc] = pa[p];
      Bs[lk + 4 * p][lc] = pb[p];
    }
    __syncthreads();
    if (k0 + 16 < k1) fetch(k0 + 16);
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      double a[4], b[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) { a[x] = static_cast<double>(As[kk][ty * 4 + x]); b[x] = static_cast<double>(Bs[kk][tx * 4 + x]); }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] += a[x] * b[y];
    }
    __syncthreads();
  }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = i0 + ty * 4 + x;
    if (i >= m.L) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int j = j0 + tx * 4 + y;
      if (j <= i) atomicAdd(m.C + static_cast<long long>(i) * m.L + j, acc[x][y]);
    }
  }
}

struct GramPrep64 {
  const double* G;  // L x L exact Gram matrix, lower triangle valid
  double* C64;      // L x L out: column-scaled Gram + tiny shift, lower triangle
  double* D;
  int L;
};

// Column scaling for the exact pass; the shift only keeps a numerically rank-deficient basis factorisable.
__global__ void __launch_bounds__(256) gram_prep64_kernel(const GramPrep64* probs) {
  const GramPrep64 p = probs[blockIdx.x];
  for (int i = threadIdx.x; i < p.L; i += 256) p.D[i] = sqrt(fmax(p.G[static_cast<long long>(i) * p.L + i], 1e-60));
  __syncthreads();
  const long long total = static_cast<long long>(p.L) * p.L;
  for (long long x = threadIdx.x; x < total; x += 256) {
    const int i = static_cast<int>(x / p.L), j = static_cast<int>(x % p.L);
    if (j > i) continue;
    p.C64[x] = (i == j) ? 1.0 + 1e-12 : p.G[x] / (p.D[i] * p.D[j]);
  }
}

struct TriInverse {
  const double* Lf;      // L x L lower Cholesky factor of the column-scaled Gram matrix (row-major)
  const double* D;       // L column norms: R^-1 = D^-1 Lf^-T
  double* X;             // L x L: X = Lf^-1 (lower triangular, upper part zero)
  __nv_bfloat16* Rhi;    // L x ld: high part of R^-1 = Lf^-T (upper triangular)
  __nv_bfloat16* Rlo;
  int L, ld;
};

// ---- blocked inverse of the lower Cholesky factor: X = Lf^-1 by recursive halving,
//   [[A, 0], [C, B]]^-1 = [[A^-1, 0], [-B^-1 C A^-1, B^-1]],
// leaves (<= 32 x 32) by forward substitution, inner nodes by two small batched fp64 GEMMs per level.

// (the pointers of TriLeaf and TriGemm are those of elements of type T, whatever their declared type: the tables
// exist once for matrices of doubles and once for the same buffers holding floats)
struct TriLeaf {
  const void* Lf;  // top-left element of the diagonal block inside the L x L factor
  void* X;         // same position inside X
  int ld, size;
};

// One warp per leaf; lane j solves column j of the block by forward substitution in shared memory.
template <typename T>
__global__ void __launch_bounds__(128) tri_leaf_kernel(const TriLeaf* leaves, int n_leaves) {
  __shared__ T blk[4][32][33];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int id = blockIdx.x * 4 + warp;
  if (id >= n_leaves) return;
  const TriLeaf lf = leaves[id];
  const T* Lf = static_cast<const T*>(lf.Lf);
  T* X = static_cast<T*>(lf.X);
  for (int i = 0; i < lf.size; ++i)
    if (lane < lf.size) blk[warp][i][lane] = Lf[static_cast<long long>(i) * lf.ld + lane];
  __syncwarp();
  if (lane < lf.size) {
    T x[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      T acc = (i == lane) ? T(1) : T(0);
      if (i < lf.size && i >= lane) {
#pragma unroll
        for (int k = 0; k < 32; ++k)
          if (k < i && k >= lane) acc -= blk[warp][i][k] * x[k];
        acc /= blk[warp][i][i];
      } else {
        acc = T(0);
      }
      x[i] = acc;
      if (i < lf.size) X[static_cast<long long>(i) * lf.ld + lane] = acc;
    }
  }
}

struct TriGemm {
  const void* A;  // m x k
  const void* B;  // k x n
  void* C;        // m x n = (negate ? -1 : 1) * A B
  int lda, ldb, ldc, m, n, k, negate;
};

// Batched small GEMM: blockIdx.z selects the problem, (blockIdx.y, blockIdx.x) a 64 x 64 tile of it.
template <typename T>
__global__ void __launch_bounds__(256) tri_gemm_kernel(const TriGemm* probs) {
  __shared__ T As[16][64 + 1];
  __shared__ T Bs[16][64 + 1];
  const TriGemm g = probs[blockIdx.z];
  const T* gA = static_cast<const T*>(g.A);
  const T* gB = static_cast<const T*>(g.B);
  T* gC = static_cast<T*>(g.C);
  const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
  if (i0 >= g.m || j0 >= g.n) return;
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  T acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = T(0);
  for (int k0 = 0; k0 < g.k; k0 += 16) {
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      const int kk = t & 15, i = (t >> 4) + 16 * p;  // A: k contiguous
      As[kk][i] = (i0 + i < g.m && k0 + kk < g.k) ? gA[static_cast<long long>(i0 + i) * g.lda + k0 + kk] : T(0);
      const int j = t & 63, kb = (t >> 6) + 4 * p;   // B: n contiguous
      Bs[kb][j] = (j0 + j < g.n && k0 + kb < g.k) ? gB[static_cast<long long>(k0 + kb) * g.ldb + j0 + j] : T(0);
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      T a[4], b[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) { a[x] = As[kk][ty * 4 + x]; b[x] = Bs[kk][tx * 4 + x]; }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] += a[x] * b[y];
    }
    __syncthreads();
  }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = i0 + ty * 4 + x;
    if (i >= g.m) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int j = j0 + tx * 4 + y;
      if (j < g.n) gC[static_cast<long long>(i) * g.ldc + j] = g.negate ? -acc[x][y] : acc[x][y];
    }
  }
}

// R^-1 = D^-1 X^T (upper triangular) split into two bf16 parts; blockIdx.x = matrix, blockIdx.y = share of its entries.
template <typename T>
__global__ void __launch_bounds__(256) tri_convert_kernel(const TriInverse* probs) {
  const TriInverse p = probs[blockIdx.x];
  const T* X = reinterpret_cast<const T*>(p.X);
  const long long total = static_cast<long long>(p.L) * p.L;
  for (long long x = blockIdx.y * 256 + threadIdx.x; x < total; x += 256ll * gridDim.y) {
    const int j = static_cast<int>(x / p.L), i = static_cast<int>(x % p.L);  // entry (j, i) of R^-1
    const double v = (i >= j) ? static_cast<double>(X[static_cast<long long>(i) * p.L + j]) / p.D[j] : 0.0;
    const float f = static_cast<float>(fmin(fmax(v, -1e30), 1e30));
    const __nv_bfloat16 h = __float2bfloat16_rn(f);
    p.Rhi[static_cast<long long>(j) * p.ld + i] = h;
    p.Rlo[static_cast<long long>(j) * p.ld + i] = __float2bfloat16_rn(f - __bfloat162float(h));
  }
}

// Second-order orthonormalisation of a basis that is orthonormal to first order already: with C = Q^T Q = I + E,
// Q (I - E / 2) has Q^T Q = I + O(E^2).  C comes from the tensor cores (its error, about 1e-7 on an entry for columns
// of unit norm, is what is left of E afterwards); S = I - E / 2 = 1.5 I - C / 2 is written in two bf16 parts where the
// product Q = Y R^-1 expects R^-1.  blockIdx.x = matrix, blockIdx.y = share of its entries.
__global__ void __launch_bounds__(256) newton_prep_kernel(const GramPrep* preps, const TriInverse* tris) {
  const GramPrep g = preps[blockIdx.x];
  const TriInverse t = tris[blockIdx.x];
  const long long total = static_cast<long long>(g.L) * g.L;
  for (long long x = blockIdx.y * 256 + threadIdx.x; x < total; x += 256ll * gridDim.y) {
    const int j = static_cast<int>(x / g.L), i = static_cast<int>(x % g.L);
    const float c = 0.5f * (g.C32[x] + g.C32[static_cast<long long>(i) * g.L + j]);
    const float f = (i == j) ? 1.5f - 0.5f * c : -0.5f * c;
    const __nv_bfloat16 h = __float2bfloat16_rn(f);
    t.Rhi[static_cast<long long>(j) * t.ld + i] = h;
    t.Rlo[static_cast<long long>(j) * t.ld + i] = __float2bfloat16_rn(f - __bfloat162float(h));
  }
}

// Scale every column of Y (rows x L, fp32) to unit norm, the norm summed in fp64.  The products of the refresh go
// through operands split in two bf16 parts; the rounding of the diagonal of a triangular factor or of a rotation
// (a relative 2^-17) scales a whole column, which is the largest part of what the last product leaves of
// non-orthonormality.  Two kernels: partial sums of squares per strip of 32 columns and chunk of rows (added to
// `sums` with fp64 atomics; `sums` is cleared beforehand), then the scaling.  Block (32, 8): blockIdx.x = strip of
// 32 columns, blockIdx.y = matrix, blockIdx.z = chunk of kNormRows rows.
struct NormJob {
  float* Y;
  double* sums;   // L sums of squares
  int rows, L;
};
constexpr int kNormRows = 1024;

__global__ void __launch_bounds__(256) column_sumsq_kernel(const NormJob* jobs) {
  __shared__ double part[8][33];
  const NormJob jb = jobs[blockIdx.y];
  const int col = blockIdx.x * 32 + threadIdx.x;
  const int r0 = blockIdx.z * kNormRows;
  if (blockIdx.x * 32 >= jb.L || r0 >= jb.rows) return;
  const int r1 = min(jb.rows, r0 + kNormRows);
  double s = 0.0;
  if (col < jb.L)
    for (int r = r0 + threadIdx.y; r < r1; r += 8) {
      const double v = static_cast<double>(jb.Y[static_cast<long long>(r) * jb.L + col]);
      s += v * v;
    }
  part[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && col < jb.L) {
    double t = 0.0;
#pragma unroll
    for (int g = 0; g < 8; ++g) t += part[g][threadIdx.x];
    atomicAdd(jb.sums + col, t);
  }
}

__global__ void __launch_bounds__(256) column_scale_kernel(const NormJob* jobs) {
  const NormJob jb = jobs[blockIdx.y];
  const int col = blockIdx.x * 32 + threadIdx.x;
  const int r0 = blockIdx.z * kNormRows;
  if (col >= jb.L || r0 >= jb.rows) return;
  const int r1 = min(jb.rows, r0 + kNormRows);
  const double t = jb.sums[col];
  const float f = t > 0.0 ? static_cast<float>(1.0 / sqrt(t)) : 0.f;
  for (int r = r0 + threadIdx.y; r < r1; r += 8) jb.Y[static_cast<long long>(r) * jb.L + col] *= f;
}

constexpr int kTriMaxLevels = 12;

// ------------------------------------------------------------------------------------------ plan

enum RefreshGemm { RG_Y_FROM_Z = 0, RG_Z_FROM_Y, RG_GRAM_Y, RG_GRAM_Z, RG_APPLY_Y, RG_COUNT };
enum RefreshMap { RM_G_A = 0, RM_G_MN, RM_Z_B, RM_Z_B_LO, RM_Y_B, RM_Y_B_LO, RM_Y_A, RM_Y_A_LO,
                  RM_RINV, RM_RINV_LO, RM_COUNT };

struct RefreshMat {
  int M, N, L, ldl;
  float *Yf, *Zf;                       // fp32 GEMM outputs (M x L, N x L)
  __nv_bfloat16 *Yhi, *Ylo, *Zhi, *Zlo; // bf16 parts of the iterates (rows x ldl)
  float* C32;                           // L x L
  double *C64, *X64, *T64;              // L x L each
  double* D;                            // L
  __nv_bfloat16 *Rhi, *Rlo;             // L x ldl
};

constexpr int kRefBN = 128;
constexpr int kRefStages1 = 4;  // NA = 1, NB = 2: 48 KB per stage
constexpr int kRefStages0 = 6;  // NA = 1, NB = 1: 32 KB per stage
constexpr int kRefStages2 = 3;  // NA = 2, NB = 2: 64 KB per stage

struct RefreshPlan {
  bool ready = false;
  size_t device_bytes = 0;
  EncodeTiledFn encode = nullptr;
  int n = 0;
  std::vector<RefreshMat> mats;
  std::vector<CUtensorMap> h_maps;  // RM_COUNT per matrix
  std::vector<const void*> last_G;
  char* buf = nullptr;
  char* tri_tables[2] = {nullptr, nullptr};
  CUtensorMap* d_maps = nullptr;
  TcProblem* d_probs[RG_COUNT] = {};
  TcTile* d_tiles[RG_COUNT] = {};
  int n_tiles[RG_COUNT] = {};
  int grid[RG_COUNT] = {};
  std::vector<int> atomic_mats[RG_COUNT];  // matrices whose K is split for this GEMM (output must be zeroed)
  // buffers to clear before GEMM kind g (the outputs of atomic_mats[g]); entry RG_COUNT: every matrix's X64
  ZeroJob* d_zero[RG_COUNT + 1] = {};
  int n_zero[RG_COUNT + 1] = {};
  char* zero_tables = nullptr;
  GramPrep* d_prep = nullptr;
  CholProblem* d_chol = nullptr;
  CholProblem* d_chol_sorted = nullptr;  // the same problems, widest first (for the one-CTA-per-matrix kernel)
  int l_max = 0;  // largest basis width L of the set
  TriInverse* d_tri = nullptr;
  TriLeaf* d_leaves[2] = {nullptr, nullptr};   // [0]: the buffers hold doubles, [1]: floats
  int n_leaves = 0;
  TriGemm* d_tg1[2][kTriMaxLevels] = {};
  TriGemm* d_tg2[2][kTriMaxLevels] = {};
  int n_tg[kTriMaxLevels] = {};
  int tg_max[kTriMaxLevels] = {};
  int tri_levels = 0;
  SplitJob* d_split_y = nullptr;
  // the matrices whose product with G splits K (their result arrives as fp32 and is split afterwards; all others
  // leave the product as bf16 parts already)
  SplitJob* d_split_y_rest = nullptr;
  SplitJob* d_split_z_rest = nullptr;
  int n_split_y_rest = 0, n_split_z_rest = 0;
  SyrkMat* d_syrk_mats = nullptr;
  SyrkTile* d_syrk_tiles = nullptr;
  int n_syrk_tiles = 0;
  GramPrep64* d_prep64 = nullptr;
  SplitJob* d_split_z = nullptr;
  // Rayleigh-Ritz rotation: the Jacobi kernels work in the T64 (X, fp32) and X64 (V, fp64) buffers
  JacobiMat* d_jac = nullptr;
  JacobiInit* d_jac_init = nullptr;
  JacobiOut* d_jac_out = nullptr;
  NormJob* d_norm = nullptr;
  FillJob* d_fill = nullptr;   // the random start Z = Omega of every matrix
  ZeroJob* d_zero_d = nullptr;   // clears every matrix's D (as 16-byte words)
  int m_max = 0;                 // most rows among the matrices
};

inline void refresh_plan_destroy(RefreshPlan& plan) {
  if (plan.buf) cudaFree(plan.buf);
  for (int set = 0; set < 2; ++set)
    if (plan.tri_tables[set]) cudaFree(plan.tri_tables[set]);
  if (plan.zero_tables) cudaFree(plan.zero_tables);
  plan.zero_tables = nullptr;
  plan.buf = nullptr;
  plan.tri_tables[0] = plan.tri_tables[1] = nullptr;
  plan.ready = false;
}

inline ngalore_status refresh_plan_create(RefreshPlan& plan, const std::vector<MatDesc>& mats,
                                          const std::vector<float*>& Yf, const std::vector<float*>& Zf, int sm_count,
                                          int ritz_columns) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr)
    return NGALORE_ERR_CUDA;
  plan.encode = reinterpret_cast<EncodeTiledFn>(fn);
  const int n = static_cast<int>(mats.size());
  plan.n = n;
  plan.mats.resize(n);
  plan.last_G.assign(n, nullptr);

  // ---- tile and problem tables (host)
  std::vector<TcProblem> probs[RG_COUNT];
  std::vector<TcTile> tiles[RG_COUNT];
  for (int g = 0; g < RG_COUNT; ++g) probs[g].resize(n);
  auto add_tiles = [&](int g, int i, int out_rows, int out_cols, int K, long long target_kb) {
    const int kb_total = (K + kTcBK - 1) / kTcBK;
    int splits = static_cast<int>((kb_total + target_kb - 1) / target_kb);
    if (splits < 1) splits = 1;
    const int kb_per = (kb_total + splits - 1) / splits;
    splits = (kb_total + kb_per - 1) / kb_per;
    if (splits > 1) plan.atomic_mats[g].push_back(i);
    for (int n0 = 0; n0 < out_cols; n0 += kRefBN)
      for (int sp = 0; sp < splits; ++sp)
        for (int m0 = 0; m0 < out_rows; m0 += kTcBM) {
          const int kb0 = sp * kb_per;
          const int kbn = std::min(kb_per, kb_total - kb0);
          tiles[g].push_back(TcTile{i, m0, n0, kb0 * kTcBK, kbn, splits > 1 ? 1 : 0, out_rows, out_cols});
        }
  };

  // ---- device buffer layout
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 255) / 256 * 256; return o; };
  struct Offs { size_t Yhi, Ylo, Zhi, Zlo, C32, C64, X64, T64, D, Rhi, Rlo; };
  std::vector<Offs> offs(n);
  for (int i = 0; i < n; ++i) {
    RefreshMat& m = plan.mats[i];
    m.M = mats[i].M; m.N = mats[i].N; m.L = mats[i].rp; m.ldl = (m.L + 7) / 8 * 8;
    m.Yf = Yf[i]; m.Zf = Zf[i];
    offs[i].Yhi = take(sizeof(__nv_bfloat16) * m.M * m.ldl);
    offs[i].Ylo = take(sizeof(__nv_bfloat16) * m.M * m.ldl);
    offs[i].Zhi = take(sizeof(__nv_bfloat16) * m.N * m.ldl);
    offs[i].Zlo = take(sizeof(__nv_bfloat16) * m.N * m.ldl);
    offs[i].C32 = take(sizeof(float) * m.L * m.L);
    offs[i].C64 = take(sizeof(double) * m.L * m.L);
    offs[i].X64 = take(sizeof(double) * m.L * m.L);
    offs[i].T64 = take(sizeof(double) * m.L * m.L);
    offs[i].D = take(sizeof(double) * m.L);
    offs[i].Rhi = take(sizeof(__nv_bfloat16) * m.L * m.ldl);
    offs[i].Rlo = take(sizeof(__nv_bfloat16) * m.L * m.ldl);
  }
  const size_t o_maps = take(sizeof(CUtensorMap) * RM_COUNT * n);
  size_t o_probs[RG_COUNT], o_tiles[RG_COUNT];

  // work estimate for the split-K targets: per GEMM kind, k-blocks per CTA if perfectly balanced
  for (int g = 0; g < RG_COUNT; ++g) {
    long long total_kb = 0;
    for (int i = 0; i < n; ++i) {
      const RefreshMat& m = plan.mats[i];
      int rows, cols, K;
      switch (g) {
        case RG_Y_FROM_Z: rows = m.M; cols = m.L; K = m.N; break;
        case RG_Z_FROM_Y: rows = m.N; cols = m.L; K = m.M; break;
        case RG_GRAM_Y: rows = m.L; cols = m.L; K = m.M; break;
        case RG_GRAM_Z: rows = m.L; cols = m.L; K = m.N; break;
        default: rows = m.M; cols = m.L; K = m.L; break;  // RG_APPLY_Y
      }
      total_kb += static_cast<long long>((rows + kTcBM - 1) / kTcBM) * ((cols + kRefBN - 1) / kRefBN) *
                  ((K + kTcBK - 1) / kTcBK);
    }
    long long target = (total_kb + sm_count - 1) / sm_count / 4;
    if (target < 16) target = 16;
    for (int i = 0; i < n; ++i) {
      const RefreshMat& m = plan.mats[i];
      int rows, cols, K;
      switch (g) {
        case RG_Y_FROM_Z: rows = m.M; cols = m.L; K = m.N; break;
        case RG_Z_FROM_Y: rows = m.N; cols = m.L; K = m.M; break;
        case RG_GRAM_Y: rows = m.L; cols = m.L; K = m.M; break;
        case RG_GRAM_Z: rows = m.L; cols = m.L; K = m.N; break;
        default: rows = m.M; cols = m.L; K = m.L; break;  // RG_APPLY_Y
      }
      add_tiles(g, i, rows, cols, K, target);
    }
    std::stable_sort(tiles[g].begin(), tiles[g].end(), [](const TcTile& a, const TcTile& b) { return a.kblocks > b.kblocks; });
    o_probs[g] = take(sizeof(TcProblem) * n);
    o_tiles[g] = take(sizeof(TcTile) * tiles[g].size());
    plan.n_tiles[g] = static_cast<int>(tiles[g].size());
    plan.grid[g] = std::min(plan.n_tiles[g], sm_count);
  }
  const size_t o_prep = take(sizeof(GramPrep) * n);
  const size_t o_chol = take(sizeof(CholProblem) * n);
  const size_t o_chol_sorted = take(sizeof(CholProblem) * n);
  const size_t o_tri = take(sizeof(TriInverse) * n);
  std::vector<SyrkTile> syrk_tiles;
  for (int i = 0; i < n; ++i) {
    const int nt = (plan.mats[i].L + 63) / 64;
    for (int k0 = 0; k0 < plan.mats[i].M; k0 += kSyrkRows)
      for (int ti = 0; ti < nt; ++ti)
        for (int tj = 0; tj <= ti; ++tj) syrk_tiles.push_back(SyrkTile{i, ti, tj, k0});
  }
  plan.n_syrk_tiles = static_cast<int>(syrk_tiles.size());
  const size_t o_syrk_m = take(sizeof(SyrkMat) * n);
  const size_t o_syrk_t = take(sizeof(SyrkTile) * syrk_tiles.size());
  const size_t o_prep64 = take(sizeof(GramPrep64) * n);
  const size_t o_sy = take(sizeof(SplitJob) * n);
  const size_t o_sz = take(sizeof(SplitJob) * n);
  const size_t o_sy_rest = take(sizeof(SplitJob) * n);
  const size_t o_sz_rest = take(sizeof(SplitJob) * n);
  const size_t o_jac = take(sizeof(JacobiMat) * n);
  const size_t o_jac_init = take(sizeof(JacobiInit) * n);
  const size_t o_jac_out = take(sizeof(JacobiOut) * n);
  const size_t o_norm = take(sizeof(NormJob) * n);
  const size_t o_fill = take(sizeof(FillJob) * n);
  const size_t o_zero_d = take(sizeof(ZeroJob) * n);
  const size_t o_jac_flags = take(sizeof(int) * kJacMaxSweeps * n);
  if (cudaMalloc(&plan.buf, off) != cudaSuccess) { plan.buf = nullptr; return NGALORE_ERR_ALLOC; }
  if (cudaMemset(plan.buf, 0, off) != cudaSuccess) return NGALORE_ERR_CUDA;
  plan.device_bytes = off;

  std::vector<GramPrep> prep(n);
  std::vector<CholProblem> chol(n);
  plan.l_max = 0;
  for (const RefreshMat& m : plan.mats) plan.l_max = m.L > plan.l_max ? m.L : plan.l_max;
  std::vector<TriInverse> tri(n);
  std::vector<SplitJob> sy(n), sz(n), sy_rest, sz_rest;
  std::vector<SyrkMat> syrk_m(n);
  std::vector<GramPrep64> prep64(n);
  std::vector<JacobiMat> jac(n);
  std::vector<JacobiInit> jac_init(n);
  std::vector<JacobiOut> jac_out(n);
  std::vector<NormJob> norm(n);
  plan.h_maps.resize(static_cast<size_t>(RM_COUNT) * n);
  std::memset(plan.h_maps.data(), 0, sizeof(CUtensorMap) * plan.h_maps.size());
  for (int i = 0; i < n; ++i) {
    RefreshMat& m = plan.mats[i];
    m.Yhi = reinterpret_cast<__nv_bfloat16*>(plan.buf + offs[i].Yhi);
    m.Ylo = reinterpret_cast<__nv_bfloat16*>(plan.buf + offs[i].Ylo);
    m.Zhi = reinterpret_cast<__nv_bfloat16*>(plan.buf + offs[i].Zhi);
    m.Zlo = reinterpret_cast<__nv_bfloat16*>(plan.buf + offs[i].Zlo);
    m.C32 = reinterpret_cast<float*>(plan.buf + offs[i].C32);
    m.C64 = reinterpret_cast<double*>(plan.buf + offs[i].C64);
    m.X64 = reinterpret_cast<double*>(plan.buf + offs[i].X64);
    m.T64 = reinterpret_cast<double*>(plan.buf + offs[i].T64);
    m.D = reinterpret_cast<double*>(plan.buf + offs[i].D);
    m.Rhi = reinterpret_cast<__nv_bfloat16*>(plan.buf + offs[i].Rhi);
    m.Rlo = reinterpret_cast<__nv_bfloat16*>(plan.buf + offs[i].Rlo);
    prep[i] = GramPrep{m.C32, m.C64, m.D, m.L};
    chol[i] = CholProblem{m.C64, m.L, 0, 0.0};
    tri[i] = TriInverse{m.C64, m.D, m.X64, m.Rhi, m.Rlo, m.L, m.ldl};
    syrk_m[i] = SyrkMat{m.Yf, m.X64, m.M, m.L};
    prep64[i] = GramPrep64{m.X64, m.C64, m.D, m.L};
    sy[i] = SplitJob{m.Yf, m.Yhi, m.Ylo, static_cast<long long>(m.M) * m.L, m.L, m.ldl};
    sz[i] = SplitJob{m.Zf, m.Zhi, m.Zlo, static_cast<long long>(m.N) * m.L, m.L, m.ldl};
    if (std::find(plan.atomic_mats[RG_Y_FROM_Z].begin(), plan.atomic_mats[RG_Y_FROM_Z].end(), i) != plan.atomic_mats[RG_Y_FROM_Z].end())
      sy_rest.push_back(sy[i]);
    if (std::find(plan.atomic_mats[RG_Z_FROM_Y].begin(), plan.atomic_mats[RG_Z_FROM_Y].end(), i) != plan.atomic_mats[RG_Z_FROM_Y].end())
      sz_rest.push_back(sz[i]);
    // the Jacobi rotation keeps X (fp32) in the memory of T64 and V (fp64) in X64 (L is a multiple of 4 on this path)
    // (width of the rotated part: all of the basis, or its leading ritz_columns, kept a multiple of 4)
    const int Lj = std::min(m.L, (ritz_columns + 3) & ~3);
    jac[i] = JacobiMat{reinterpret_cast<float*>(m.T64), m.X64, Lj, Lj, jacobi_blocks(Lj),
                       reinterpret_cast<int*>(plan.buf + o_jac_flags) + kJacMaxSweeps * i};
    norm[i] = NormJob{m.Yf, m.D, m.M, m.L};   // the column-norm buffer of the orthonormalisations is free by then
    jac_init[i] = JacobiInit{m.C32, nullptr, m.L};
    jac_out[i] = JacobiOut{nullptr, 0, m.Rhi, m.Rlo, m.ldl, m.L};
    CUtensorMap* mp = &plan.h_maps[static_cast<size_t>(i) * RM_COUNT];
    const uint64_t sl = static_cast<uint64_t>(m.ldl) * 2;
    bool ok = true;
    ok &= tc_encode_2d(plan.encode, mp + RM_Z_B, m.Zhi, m.L, m.N, sl, 64, kTcBK);
    ok &= tc_encode_2d(plan.encode, mp + RM_Z_B_LO, m.Zlo, m.L, m.N, sl, 64, kTcBK);
    ok &= tc_encode_2d(plan.encode, mp + RM_Y_B, m.Yhi, m.L, m.M, sl, 64, kTcBK);
    ok &= tc_encode_2d(plan.encode, mp + RM_Y_B_LO, m.Ylo, m.L, m.M, sl, 64, kTcBK);
    ok &= tc_encode_2d(plan.encode, mp + RM_Y_A, m.Yhi, m.L, m.M, sl, kTcBK, kTcBM);
    ok &= tc_encode_2d(plan.encode, mp + RM_Y_A_LO, m.Ylo, m.L, m.M, sl, kTcBK, kTcBM);
    ok &= tc_encode_2d(plan.encode, mp + RM_RINV, m.Rhi, m.L, m.L, sl, 64, kTcBK);
    ok &= tc_encode_2d(plan.encode, mp + RM_RINV_LO, m.Rlo, m.L, m.L, sl, 64, kTcBK);
    if (!ok) return NGALORE_ERR_CUDA;
    const int base = i * RM_COUNT;
    probs[RG_Y_FROM_Z][i] = TcProblem{m.Yf, m.M, m.L, m.L, base + RM_G_A, base + RM_Z_B, 0};
    probs[RG_Z_FROM_Y][i] = TcProblem{m.Zf, m.N, m.L, m.L, base + RM_G_MN, base + RM_Y_B, 0};
    {
      const std::vector<int>& ay = plan.atomic_mats[RG_Y_FROM_Z];
      const std::vector<int>& az = plan.atomic_mats[RG_Z_FROM_Y];
      if (std::find(ay.begin(), ay.end(), i) == ay.end()) {
        probs[RG_Y_FROM_Z][i].ld16 = m.ldl; probs[RG_Y_FROM_Z][i].out_hi = m.Yhi; probs[RG_Y_FROM_Z][i].out_lo = m.Ylo;
      }
      if (std::find(az.begin(), az.end(), i) == az.end()) {
        probs[RG_Z_FROM_Y][i].ld16 = m.ldl; probs[RG_Z_FROM_Y][i].out_hi = m.Zhi; probs[RG_Z_FROM_Y][i].out_lo = m.Zlo;
      }
    }
    probs[RG_GRAM_Y][i] = TcProblem{m.C32, m.L, m.L, m.L, base + RM_Y_B, base + RM_Y_B, 0};
    probs[RG_GRAM_Z][i] = TcProblem{m.C32, m.L, m.L, m.L, base + RM_Z_B, base + RM_Z_B, 0};
    probs[RG_APPLY_Y][i] = TcProblem{m.Yf, m.M, m.L, m.L, base + RM_Y_A, base + RM_RINV, 0};
  }
  // ---- tables of the blocked triangular inverse, for the buffers holding doubles (set 0) and floats (set 1)
  for (int set = 0; set < 2; ++set) {
    const size_t esz = set == 0 ? sizeof(double) : sizeof(float);
    std::vector<TriLeaf> leaves;
    std::vector<TriGemm> g1[kTriMaxLevels], g2[kTriMaxLevels];
    int max_level = 0;
    for (int i = 0; i < n; ++i) {
      const RefreshMat& m = plan.mats[i];
      // returns the height of the node covering [lo, hi)
      struct Rec {
        size_t esz;
        void* at(double* buf, const RefreshMat& m, int row, int col) const {
          return reinterpret_cast<char*>(buf) + esz * (static_cast<size_t>(row) * m.L + col);
        }
        int go(const RefreshMat& m, int lo, int hi, std::vector<TriLeaf>& leaves, std::vector<TriGemm>* g1,
               std::vector<TriGemm>* g2) const {
          const int len = hi - lo;
          if (len <= 32) {
            leaves.push_back(TriLeaf{at(m.C64, m, lo, lo), at(m.X64, m, lo, lo), m.L, len});
            return 0;
          }
          const int mid = lo + ((len / 2 + 31) / 32) * 32;
          const int ha = go(m, lo, mid, leaves, g1, g2), hb = go(m, mid, hi, leaves, g1, g2);
          const int h = (ha > hb ? ha : hb) + 1;
          // T = C A^-1 with C = Lf[mid:hi, lo:mid];  X[mid:hi, lo:mid] = -B^-1 T
          void* T = at(m.T64, m, mid, lo);
          g1[h].push_back(TriGemm{at(m.C64, m, mid, lo), at(m.X64, m, lo, lo), T, m.L, m.L, m.L, hi - mid, mid - lo,
                                  mid - lo, 0});
          g2[h].push_back(TriGemm{at(m.X64, m, mid, mid), T, at(m.X64, m, mid, lo), m.L, m.L, m.L, hi - mid, mid - lo,
                                  hi - mid, 1});
          return h;
        }
      };
      const int h = Rec{esz}.go(m, 0, m.L, leaves, g1, g2);
      if (h > max_level) max_level = h;
    }
    if (max_level >= kTriMaxLevels) return NGALORE_ERR_INVALID_ARG;
    plan.tri_levels = max_level;
    plan.n_leaves = static_cast<int>(leaves.size());
    size_t bytes = sizeof(TriLeaf) * leaves.size();
    for (int h = 1; h <= max_level; ++h) bytes += 2 * ((sizeof(TriGemm) * g1[h].size() + 255) / 256 * 256);
    bytes = (bytes + 255) / 256 * 256 + 256;
    char* tb = nullptr;
    if (cudaMalloc(&tb, bytes) != cudaSuccess) return NGALORE_ERR_ALLOC;
    plan.tri_tables[set] = tb;
    plan.device_bytes += bytes;
    size_t o = 0;
    plan.d_leaves[set] = reinterpret_cast<TriLeaf*>(tb);
    if (cudaMemcpy(tb, leaves.data(), sizeof(TriLeaf) * leaves.size(), cudaMemcpyHostToDevice) != cudaSuccess) return NGALORE_ERR_CUDA;
    o = (sizeof(TriLeaf) * leaves.size() + 255) / 256 * 256;
    for (int h = 1; h <= max_level; ++h) {
      const size_t sz = sizeof(TriGemm) * g1[h].size();
      plan.n_tg[h] = static_cast<int>(g1[h].size());
      int mx = 1;
      for (const TriGemm& g : g1[h]) { if (g.m > mx) mx = g.m; if (g.n > mx) mx = g.n; }
      plan.tg_max[h] = mx;
      plan.d_tg1[set][h] = reinterpret_cast<TriGemm*>(tb + o);
      if (sz && cudaMemcpy(tb + o, g1[h].data(), sz, cudaMemcpyHostToDevice) != cudaSuccess) return NGALORE_ERR_CUDA;
      o += (sz + 255) / 256 * 256;
      plan.d_tg2[set][h] = reinterpret_cast<TriGemm*>(tb + o);
      if (sz && cudaMemcpy(tb + o, g2[h].data(), sz, cudaMemcpyHostToDevice) != cudaSuccess) return NGALORE_ERR_CUDA;
      o += (sz + 255) / 256 * 256;
    }
  }
  plan.d_maps = reinterpret_cast<CUtensorMap*>(plan.buf + o_maps);
  for (int g = 0; g < RG_COUNT; ++g) {
    plan.d_probs[g] = reinterpret_cast<TcProblem*>(plan.buf + o_probs[g]);
    plan.d_tiles[g] = reinterpret_cast<TcTile*>(plan.buf + o_tiles[g]);
    if (cudaMemcpy(plan.d_probs[g], probs[g].data(), sizeof(TcProblem) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(plan.d_tiles[g], tiles[g].data(), sizeof(TcTile) * tiles[g].size(), cudaMemcpyHostToDevice) != cudaSuccess)
      return NGALORE_ERR_CUDA;
  }
  plan.d_prep = reinterpret_cast<GramPrep*>(plan.buf + o_prep);
  plan.d_chol = reinterpret_cast<CholProblem*>(plan.buf + o_chol);
  plan.d_chol_sorted = reinterpret_cast<CholProblem*>(plan.buf + o_chol_sorted);
  {
    std::vector<CholProblem> sorted(chol);
    std::stable_sort(sorted.begin(), sorted.end(), [](const CholProblem& a, const CholProblem& b) { return a.L > b.L; });
    if (cudaMemcpy(plan.d_chol_sorted, sorted.data(), sizeof(CholProblem) * n, cudaMemcpyHostToDevice) != cudaSuccess)
      return NGALORE_ERR_CUDA;
    if (cudaFuncSetAttribute(chol_cta_kernel<double>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(chol_cta_smem_bytes<double>(plan.l_max))) != cudaSuccess ||
        cudaFuncSetAttribute(chol_cta_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(chol_cta_smem_bytes<float>(plan.l_max))) != cudaSuccess)
      return NGALORE_ERR_CUDA;
  }
  plan.d_tri = reinterpret_cast<TriInverse*>(plan.buf + o_tri);
  plan.d_split_y = reinterpret_cast<SplitJob*>(plan.buf + o_sy);
  plan.d_syrk_mats = reinterpret_cast<SyrkMat*>(plan.buf + o_syrk_m);
  plan.d_syrk_tiles = reinterpret_cast<SyrkTile*>(plan.buf + o_syrk_t);
  plan.d_prep64 = reinterpret_cast<GramPrep64*>(plan.buf + o_prep64);
  plan.d_split_z = reinterpret_cast<SplitJob*>(plan.buf + o_sz);
  plan.d_split_y_rest = reinterpret_cast<SplitJob*>(plan.buf + o_sy_rest);
  plan.d_split_z_rest = reinterpret_cast<SplitJob*>(plan.buf + o_sz_rest);
  plan.n_split_y_rest = static_cast<int>(sy_rest.size());
  plan.n_split_z_rest = static_cast<int>(sz_rest.size());
  plan.d_jac = reinterpret_cast<JacobiMat*>(plan.buf + o_jac);
  plan.d_jac_init = reinterpret_cast<JacobiInit*>(plan.buf + o_jac_init);
  plan.d_jac_out = reinterpret_cast<JacobiOut*>(plan.buf + o_jac_out);
  plan.d_norm = reinterpret_cast<NormJob*>(plan.buf + o_norm);
  plan.d_fill = reinterpret_cast<FillJob*>(plan.buf + o_fill);
  {
    std::vector<FillJob> fill(n);
    for (int i = 0; i < n; ++i) fill[i] = FillJob{plan.mats[i].Zf, static_cast<long long>(plan.mats[i].N) * plan.mats[i].L};
    if (cudaMemcpy(plan.d_fill, fill.data(), sizeof(FillJob) * n, cudaMemcpyHostToDevice) != cudaSuccess) return NGALORE_ERR_CUDA;
  }
  plan.d_zero_d = reinterpret_cast<ZeroJob*>(plan.buf + o_zero_d);
  {
    std::vector<ZeroJob> zd(n);
    for (int i = 0; i < n; ++i) {
      zd[i] = ZeroJob{reinterpret_cast<float4*>(plan.mats[i].D), static_cast<long long>(plan.mats[i].L) * 8 / 16};  // L is a multiple of 4
      plan.m_max = std::max(plan.m_max, plan.mats[i].M);
    }
    if (cudaMemcpy(plan.d_zero_d, zd.data(), sizeof(ZeroJob) * n, cudaMemcpyHostToDevice) != cudaSuccess) return NGALORE_ERR_CUDA;
  }
  if (cudaMemcpy(plan.d_prep, prep.data(), sizeof(GramPrep) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_chol, chol.data(), sizeof(CholProblem) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_tri, tri.data(), sizeof(TriInverse) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_syrk_mats, syrk_m.data(), sizeof(SyrkMat) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_syrk_tiles, syrk_tiles.data(), sizeof(SyrkTile) * syrk_tiles.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_prep64, prep64.data(), sizeof(GramPrep64) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_split_y, sy.data(), sizeof(SplitJob) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_split_z, sz.data(), sizeof(SplitJob) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_split_y_rest, sy_rest.data(), sizeof(SplitJob) * sy_rest.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_split_z_rest, sz_rest.data(), sizeof(SplitJob) * sz_rest.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_jac, jac.data(), sizeof(JacobiMat) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_jac_init, jac_init.data(), sizeof(JacobiInit) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_jac_out, jac_out.data(), sizeof(JacobiOut) * n, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(plan.d_norm, norm.data(), sizeof(NormJob) * n, cudaMemcpyHostToDevice) != cudaSuccess)
    return NGALORE_ERR_CUDA;

  // ---- tables of buffers to clear
  {
    std::vector<ZeroJob> jobs;
    int first[RG_COUNT + 2];
    for (int g = 0; g <= RG_COUNT; ++g) {
      first[g] = static_cast<int>(jobs.size());
      if (g == RG_COUNT) {
        for (const RefreshMat& m : plan.mats)
          jobs.push_back(ZeroJob{reinterpret_cast<float4*>(m.X64), static_cast<long long>(m.L) * m.L * 8 / 16});
        continue;
      }
      for (int i : plan.atomic_mats[g]) {
        const RefreshMat& m = plan.mats[i];
        float* out; long long bytes;
        switch (g) {
          case RG_Y_FROM_Z: case RG_APPLY_Y: out = m.Yf; bytes = 4ll * m.M * m.L; break;
          case RG_Z_FROM_Y: out = m.Zf; bytes = 4ll * m.N * m.L; break;
          default: out = m.C32; bytes = 4ll * m.L * m.L; break;
        }
        jobs.push_back(ZeroJob{reinterpret_cast<float4*>(out), bytes / 16});  // L is a multiple of 4
      }
    }
    first[RG_COUNT + 1] = static_cast<int>(jobs.size());
    if (cudaMalloc(&plan.zero_tables, sizeof(ZeroJob) * (jobs.size() + 1)) != cudaSuccess) {
      plan.zero_tables = nullptr;
      return NGALORE_ERR_ALLOC;
    }
    if (!jobs.empty() && cudaMemcpy(plan.zero_tables, jobs.data(), sizeof(ZeroJob) * jobs.size(), cudaMemcpyHostToDevice) != cudaSuccess)
      return NGALORE_ERR_CUDA;
    for (int g = 0; g <= RG_COUNT; ++g) {
      plan.d_zero[g] = reinterpret_cast<ZeroJob*>(plan.zero_tables) + first[g];
      plan.n_zero[g] = first[g + 1] - first[g];
    }
    plan.device_bytes += sizeof(ZeroJob) * (jobs.size() + 1);
  }

  using L1 = TcSmem<kRefBN, 1, 2, kRefStages1, 4>;
  using L2 = TcSmem<kRefBN, 2, 2, kRefStages2, 4>;
  using L0 = TcSmem<kRefBN, 1, 1, kRefStages0, 4>;
  if (cudaFuncSetAttribute(tc_gemm_kernel<kRefBN, 1, 1, kRefStages0, TC_EPI_STORE, 4, false>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, L0::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(tc_gemm_kernel<kRefBN, 1, 1, kRefStages0, TC_EPI_STORE, 4, true>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, L0::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(tc_gemm_kernel<kRefBN, 1, 2, kRefStages1, TC_EPI_STORE, 4, false>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, L1::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(tc_gemm_kernel<kRefBN, 1, 2, kRefStages1, TC_EPI_STORE, 4, true>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, L1::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(tc_gemm_kernel<kRefBN, 2, 2, kRefStages2, TC_EPI_STORE, 4, false>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, L2::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(tc_gemm_kernel<kRefBN, 2, 2, kRefStages2, TC_EPI_STORE, 4, true>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, L2::kTotal) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  plan.ready = true;
  return NGALORE_OK;
}


// high_only: the products with G take only the high bf16 part of the basis (half the tensor-core work; the basis
// then enters with 8 bits instead of 16, which the early sweeps of the iteration do not notice).
inline ngalore_status refresh_tc_gemm(RefreshPlan& plan, int g, Ctrl* d_ctrl, cudaStream_t stream, int64_t* launches,
                                      bool high_only = false) {
  // outputs that several K slices accumulate into start from zero
  if (plan.n_zero[g] > 0) {
    zero_jobs_kernel<<<dim3(32, plan.n_zero[g]), 256, 0, stream>>>(plan.d_zero[g]);
    *launches += 1;
  }
  using L1 = TcSmem<kRefBN, 1, 2, kRefStages1, 4>;
  using L2 = TcSmem<kRefBN, 2, 2, kRefStages2, 4>;
  const int threads = 64 + 32 * 4;
  using L0 = TcSmem<kRefBN, 1, 1, kRefStages0, 4>;
  switch (g) {
    case RG_Y_FROM_Z:
      if (high_only)
        tc_gemm_kernel<kRefBN, 1, 1, kRefStages0, TC_EPI_STORE, 4, false><<<plan.grid[g], threads, L0::kTotal, stream>>>(
            plan.d_maps, plan.d_tiles[g], plan.n_tiles[g], nullptr, d_ctrl, plan.d_probs[g]);
      else
        tc_gemm_kernel<kRefBN, 1, 2, kRefStages1, TC_EPI_STORE, 4, false><<<plan.grid[g], threads, L1::kTotal, stream>>>(
            plan.d_maps, plan.d_tiles[g], plan.n_tiles[g], nullptr, d_ctrl, plan.d_probs[g]);
      break;
    case RG_Z_FROM_Y:
      if (high_only)
        tc_gemm_kernel<kRefBN, 1, 1, kRefStages0, TC_EPI_STORE, 4, true><<<plan.grid[g], threads, L0::kTotal, stream>>>(
            plan.d_maps, plan.d_tiles[g], plan.n_tiles[g], nullptr, d_ctrl, plan.d_probs[g]);
      else
        tc_gemm_kernel<kRefBN, 1, 2, kRefStages1, TC_EPI_STORE, 4, true><<<plan.grid[g], threads, L1::kTotal, stream>>>(
            plan.d_maps, plan.d_tiles[g], plan.n_tiles[g], nullptr, d_ctrl, plan.d_probs[g]);
      break;
    case RG_GRAM_Y:
    case RG_GRAM_Z:
      tc_gemm_kernel<kRefBN, 2, 2, kRefStages2, TC_EPI_STORE, 4, true><<<plan.grid[g], threads, L2::kTotal, stream>>>(
          plan.d_maps, plan.d_tiles[g], plan.n_tiles[g], nullptr, d_ctrl, plan.d_probs[g]);
      break;
    default:
      tc_gemm_kernel<kRefBN, 2, 2, kRefStages2, TC_EPI_STORE, 4, false><<<plan.grid[g], threads, L2::kTotal, stream>>>(
          plan.d_maps, plan.d_tiles[g], plan.n_tiles[g], nullptr, d_ctrl, plan.d_probs[g]);
      break;
  }
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

// X = Lf^-1 for every matrix (blocked), then R^-1 = D^-1 X^T in two bf16 parts.  T: what the buffers hold.
template <typename T>
inline ngalore_status refresh_tc_tri_inverse(RefreshPlan& plan, cudaStream_t stream, int64_t* launches) {
  constexpr int set = sizeof(T) == 8 ? 0 : 1;
  zero_jobs_kernel<<<dim3(32, plan.n_zero[RG_COUNT]), 256, 0, stream>>>(plan.d_zero[RG_COUNT]);
  *launches += 1;
  tri_leaf_kernel<T><<<(plan.n_leaves + 3) / 4, 128, 0, stream>>>(plan.d_leaves[set], plan.n_leaves);
  *launches += 1;
  for (int h = 1; h <= plan.tri_levels; ++h) {
    if (plan.n_tg[h] == 0) continue;
    const int tiles = (plan.tg_max[h] + 63) / 64;
    tri_gemm_kernel<T><<<dim3(tiles, tiles, plan.n_tg[h]), 256, 0, stream>>>(plan.d_tg1[set][h]);
    tri_gemm_kernel<T><<<dim3(tiles, tiles, plan.n_tg[h]), 256, 0, stream>>>(plan.d_tg2[set][h]);
    *launches += 2;
  }
  tri_convert_kernel<T><<<dim3(plan.n, 8), 256, 0, stream>>>(plan.d_tri);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

// after_product: the iterate has just left a product with G, which wrote the bf16 parts itself except for the
// matrices whose K it splits.
inline ngalore_status refresh_tc_split(RefreshPlan& plan, bool y_side, cudaStream_t stream, int64_t* launches,
                                       bool after_product = false) {
  const SplitJob* jobs = y_side ? plan.d_split_y : plan.d_split_z;
  int n_jobs = plan.n;
  if (after_product) {
    jobs = y_side ? plan.d_split_y_rest : plan.d_split_z_rest;
    n_jobs = y_side ? plan.n_split_y_rest : plan.n_split_z_rest;
    if (n_jobs == 0) return NGALORE_OK;
  }
  split_hilo_grouped_kernel<<<dim3(64, n_jobs), 256, 0, stream>>>(jobs);
  *launches += 1;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

// iterate (as it leaves the product Y = G Z) -> well-conditioned basis, left both as fp32 and as its bf16 parts.
inline ngalore_status refresh_tc_orth(RefreshPlan& plan, Ctrl* d_ctrl, cudaStream_t stream, int64_t* launches,
                                      double shift_scale = 1.0) {
  ngalore_status rc;
  if ((rc = refresh_tc_split(plan, true, stream, launches, true))) return rc;
  if ((rc = refresh_tc_gemm(plan, RG_GRAM_Y, d_ctrl, stream, launches))) return rc;
  // single precision from here to R^-1: the Gram matrix has 2^-17 of relative accuracy and a shift of about 1e-2
  gram_prep_kernel<float><<<dim3(plan.n, 8), 256, 0, stream>>>(plan.d_prep, shift_scale);
  *launches += 1;
  if (chol_cta_launch<float>(plan.d_chol_sorted, plan.n, plan.l_max, stream, launches) != cudaSuccess) return NGALORE_ERR_CUDA;
  if ((rc = refresh_tc_tri_inverse<float>(plan, stream, launches))) return rc;
  if ((rc = refresh_tc_gemm(plan, RG_APPLY_Y, d_ctrl, stream, launches))) return rc;
  return refresh_tc_split(plan, true, stream, launches);
}

// Final pass: Cholesky QR of the last basis with the Gram matrix accumulated exactly in fp64 (no shift beyond
// 1e-12), Cholesky and triangular inverse in fp64; only Q = Y R^-1 goes through the tensor cores in two bf16
// parts, whose rounding averages out over the rows.  Matrices with few rows are re-done entirely in fp64 by
// the caller.
inline ngalore_status refresh_tc_final(RefreshPlan& plan, Ctrl* d_ctrl, cudaStream_t stream, int64_t* launches) {
  ngalore_status rc;
  // (the bf16 parts of the basis, which the apply below multiplies, are current: refresh_tc_orth ends with a split)
  zero_jobs_kernel<<<dim3(32, plan.n_zero[RG_COUNT]), 256, 0, stream>>>(plan.d_zero[RG_COUNT]);
  *launches += 1;
  syrk_f64_kernel<<<plan.n_syrk_tiles, 256, 0, stream>>>(plan.d_syrk_mats, plan.d_syrk_tiles);
  gram_prep64_kernel<<<plan.n, 256, 0, stream>>>(plan.d_prep64);
  *launches += 2;
  if (chol_cta_launch<double>(plan.d_chol_sorted, plan.n, plan.l_max, stream, launches) != cudaSuccess) return NGALORE_ERR_CUDA;
  if ((rc = refresh_tc_tri_inverse<double>(plan, stream, launches))) return rc;
  return refresh_tc_gemm(plan, RG_APPLY_Y, d_ctrl, stream, launches);
}

// Pass after refresh_tc_final: the basis is orthonormal to first order by then (1e-5, up to 1e-3 for a gradient of
// low numerical rank), and a Newton step with the tensor-core Gram matrix squares what is missing, down to the
// accuracy of that Gram matrix; a second exact pass gave the same at ten times the cost.
inline ngalore_status refresh_tc_refine(RefreshPlan& plan, Ctrl* d_ctrl, cudaStream_t stream, int64_t* launches) {
  ngalore_status rc;
  if ((rc = refresh_tc_split(plan, true, stream, launches))) return rc;
  if ((rc = refresh_tc_gemm(plan, RG_GRAM_Y, d_ctrl, stream, launches))) return rc;
  newton_prep_kernel<<<dim3(plan.n, 8), 256, 0, stream>>>(plan.d_prep, plan.d_tri);
  *launches += 1;
  return refresh_tc_gemm(plan, RG_APPLY_Y, d_ctrl, stream, launches);
}

// Whole-set refresh; leaves the basis in Yf.
inline ngalore_status refresh_tc_run(RefreshPlan& plan, const uint16_t* const* G, int q, unsigned long long seed,
                                     unsigned long long stream_base, Ctrl* d_ctrl, cudaStream_t stream,
                                     int64_t* launches) {
  bool changed = false;
  for (int i = 0; i < plan.n; ++i) {
    if (plan.last_G[i] != G[i]) {
      plan.last_G[i] = G[i];
      const RefreshMat& m = plan.mats[i];
      CUtensorMap* mp = &plan.h_maps[static_cast<size_t>(i) * RM_COUNT];
      if (!tc_encode_2d(plan.encode, mp + RM_G_A, G[i], m.N, m.M, static_cast<uint64_t>(m.N) * 2, kTcBK, kTcBM) ||
          !tc_encode_2d(plan.encode, mp + RM_G_MN, G[i], m.N, m.M, static_cast<uint64_t>(m.N) * 2, 64, kTcBK))
        return NGALORE_ERR_CUDA;
      changed = true;
    }
  }
  if (changed && cudaMemcpyAsync(plan.d_maps, plan.h_maps.data(), sizeof(CUtensorMap) * plan.h_maps.size(),
                                 cudaMemcpyHostToDevice, stream) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  ngalore_status rc;
  fill_normal_grouped_kernel<<<dim3(64, plan.n), 256, 0, stream>>>(plan.d_fill, seed, stream_base);
  *launches += 1;
  if (cudaGetLastError() != cudaSuccess) return NGALORE_ERR_CUDA;
  if ((rc = refresh_tc_split(plan, false, stream, launches))) return rc;
  if ((rc = refresh_tc_gemm(plan, RG_Y_FROM_Z, d_ctrl, stream, launches))) return rc;
  if ((rc = refresh_tc_orth(plan, d_ctrl, stream, launches))) return rc;
  // A sweep applies G G^T to the basis and orthonormalises the result.  Z = G^T Q is not orthonormalised in between:
  // its columns are images of orthonormal ones, and the two-part bf16 operands keep 16 bits of every entry whatever
  // the norm of its column, so the second product loses nothing that an orthonormalisation of Z would have saved
  // (measured on the 1.1B shapes: the same Ritz vectors to all printed digits, a quarter of the refresh time less).
  for (int it = 0; it < q; ++it) {
    // the first half of the sweeps multiplies with the high bf16 part of the basis only: what that rounding adds
    // (2^-9 of an entry) shrinks with every later sweep like any other component outside the dominant subspace
    // (not with fewer than four sweeps, where every one of them counts)
    const bool coarse = q >= 4 && it < q / 2;
    if ((rc = refresh_tc_gemm(plan, RG_Z_FROM_Y, d_ctrl, stream, launches, coarse))) return rc;
    if ((rc = refresh_tc_split(plan, false, stream, launches, true))) return rc;
    if ((rc = refresh_tc_gemm(plan, RG_Y_FROM_Z, d_ctrl, stream, launches, coarse))) return rc;
    if ((rc = refresh_tc_orth(plan, d_ctrl, stream, launches))) return rc;
  }
  // Exact orthonormalisation of the basis that leaves the sweeps: the basis can be ill conditioned in its weak
  // directions, so the product with the exact triangular factor leaves it orthonormal to 1e-5 .. 1e-3 only; two
  // Newton steps start from that and end at about 1e-6.  The Rayleigh-Ritz step below relies on it (it
  // solves C v = lambda v, not C v = lambda (Q^T Q) v, and what Q lacks in orthonormality goes into the Ritz vectors).
  if ((rc = refresh_tc_final(plan, d_ctrl, stream, launches))) return rc;
  if ((rc = refresh_tc_refine(plan, d_ctrl, stream, launches))) return rc;
  if ((rc = refresh_tc_refine(plan, d_ctrl, stream, launches))) return rc;
  if ((rc = refresh_tc_split(plan, true, stream, launches))) return rc;
  // Rayleigh-Ritz: Z = G^T Q, C = Z^T Z (tensor cores: its entries are good to about 2^-17 of the diagonal, far
  // finer than the gaps that decide a Ritz vector), V = eigenvectors of C (or of its leading block, see
  // ritz_jacobi.cuh), P = Q V.
  if ((rc = refresh_tc_gemm(plan, RG_Z_FROM_Y, d_ctrl, stream, launches))) return rc;
  if ((rc = refresh_tc_split(plan, false, stream, launches, true))) return rc;
  if ((rc = refresh_tc_gemm(plan, RG_GRAM_Z, d_ctrl, stream, launches))) return rc;
  jacobi_init_kernel<<<plan.n, 256, 0, stream>>>(plan.d_jac, plan.d_jac_init);
  *launches += 1;
  if (jacobi_batched_launch(plan.d_jac, plan.n, stream, launches) != cudaSuccess)
    return NGALORE_ERR_CUDA;
  jacobi_finish_kernel<<<dim3(plan.n, kJacFinishSplit), 256, 0, stream>>>(plan.d_jac, plan.d_jac_out);
  *launches += 1;
  // Q orthonormal to about 1e-6 and V orthogonal: so is their product, once its columns are scaled back to unit norm
  if ((rc = refresh_tc_gemm(plan, RG_APPLY_Y, d_ctrl, stream, launches))) return rc;
  zero_jobs_kernel<<<dim3(1, plan.n), 256, 0, stream>>>(plan.d_zero_d);
  const dim3 norm_grid((plan.l_max + 31) / 32, plan.n, (plan.m_max + kNormRows - 1) / kNormRows);
  column_sumsq_kernel<<<norm_grid, dim3(32, 8), 0, stream>>>(plan.d_norm);
  column_scale_kernel<<<norm_grid, dim3(32, 8), 0, stream>>>(plan.d_norm);
  *launches += 3;
  return cudaGetLastError() == cudaSuccess ? NGALORE_OK : NGALORE_ERR_CUDA;
}

}  // namespace ngalore
