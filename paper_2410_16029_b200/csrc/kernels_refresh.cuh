// Pieces of the subspace refresh (Sec. 1: P spans the leading left singular vectors of G,
// "updated periodically").  The refresh is a randomized subspace iteration; every application of
// G or G^T is followed by an orthonormalisation Q = Y R^-1 with R^T R = Y^T Y (Cholesky QR with
// the Gram matrix and the factorisation in fp64).
#pragma once

#include "common.cuh"

namespace ngalore {

// ---------------------------------------------------------------- random test matrix

__device__ __forceinline__ unsigned long long splitmix64(unsigned long long x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

// Standard normal entries from a counter-based hash (Box-Muller on two hashed uniforms).
__global__ void fill_normal_kernel(float* X, long long n, unsigned long long seed, unsigned long long stream_id) {
  const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (i >= n) return;
  const unsigned long long h =
      splitmix64(seed ^ splitmix64(stream_id * 0x100000001B3ull + static_cast<unsigned long long>(i)));
  const float u1 = (static_cast<float>(h >> 40) + 1.0f) * (1.0f / 16777217.0f);
  const float u2 = static_cast<float>((h >> 8) & 0xFFFFFFull) * (1.0f / 16777216.0f);
  X[i] = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
}

// The same values for a list of matrices in one launch: blockIdx.y selects the matrix (its stream of random numbers
// is stream_base + blockIdx.y), blockIdx.x strides over its entries.
struct FillJob {
  float* X;
  long long n;
};

__global__ void fill_normal_grouped_kernel(const FillJob* jobs, unsigned long long seed, unsigned long long stream_base) {
  const FillJob jb = jobs[blockIdx.y];
  const unsigned long long stream_id = stream_base + blockIdx.y;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < jb.n; i += stride) {
    const unsigned long long h =
        splitmix64(seed ^ splitmix64(stream_id * 0x100000001B3ull + static_cast<unsigned long long>(i)));
    const float u1 = (static_cast<float>(h >> 40) + 1.0f) * (1.0f / 16777217.0f);
    const float u2 = static_cast<float>((h >> 8) & 0xFFFFFFull) * (1.0f / 16777216.0f);
    jb.X[i] = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
  }
}

// ---------------------------------------------------------------- batched Cholesky (fp64, right-looking, blocked)

struct CholProblem {
  double* C;    // L x L row-major; lower triangle in, lower Cholesky factor out (C = Lf Lf^T)
  int L;
  int pad;
  double tiny;  // pivot floor, written by chol_begin_kernel
};

constexpr int kCholNB = 32;  // panel width

// Pivot floor of every matrix from its diagonal before the factorisation starts.  A pivot that is not above it
// (rank-deficient Y) is replaced by it so that the factor stays finite; the caller runs a second
// orthonormalisation pass at the end of the refresh.  One warp per matrix.
__global__ void __launch_bounds__(32) chol_begin_kernel(CholProblem* probs) {
  CholProblem& p = probs[blockIdx.x];
  double md = 0.0;
  for (int i = threadIdx.x; i < p.L; i += 32) md = fmax(md, p.C[static_cast<long long>(i) * p.L + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) md = fmax(md, __shfl_xor_sync(0xffffffffu, md, o));
  if (threadIdx.x == 0) p.tiny = fmax(md * 1e-28, 1e-300);   // never zero: a matrix of zeros still factors
}

// Panel step at column j0, one CTA per matrix: factor the diagonal block in shared memory (one warp, lane = row),
// then solve the rows below it against the block (x D^T = c, forward substitution, one thread per row).
__global__ void __launch_bounds__(256) chol_panel_kernel(const CholProblem* probs, int j0) {
  constexpr int NB = kCholNB;
  __shared__ double D[NB][NB + 1];
  const CholProblem p = probs[blockIdx.x];
  double* C = p.C;
  const int L = p.L;
  if (j0 >= L) return;
  const int tid = threadIdx.x;
  const int nbj = (L - j0 < NB) ? (L - j0) : NB;
  const double tiny = p.tiny;
  for (int x = tid; x < NB * NB; x += 256) {
    const int a = x / NB, b = x % NB;
    D[a][b] = (a < nbj && b < nbj) ? C[static_cast<long long>(j0 + a) * L + j0 + b] : 0.0;
  }
  __syncthreads();
  if (tid < 32) {
    const int lane = tid;
    for (int k = 0; k < nbj; ++k) {
      double dkk = D[k][k];
      if (!(dkk > tiny)) dkk = tiny;
      const double lkk = sqrt(dkk);
      __syncwarp();
      if (lane == k) D[k][k] = lkk;
      if (lane > k && lane < nbj) D[lane][k] /= lkk;
      __syncwarp();
      if (lane > k && lane < nbj) {
        const double lik = D[lane][k];
        for (int j = k + 1; j <= lane; ++j) D[lane][j] -= lik * D[j][k];
      }
      __syncwarp();
    }
  }
  __syncthreads();
  for (int x = tid; x < NB * NB; x += 256) {
    const int a = x / NB, b = x % NB;
    if (a < nbj && b <= a) C[static_cast<long long>(j0 + a) * L + j0 + b] = D[a][b];
  }
  for (int i = j0 + nbj + tid; i < L; i += 256) {
    double xr[NB];
    double* crow = C + static_cast<long long>(i) * L + j0;
#pragma unroll
    for (int jj = 0; jj < NB; ++jj) {
      if (jj < nbj) {
        double a = crow[jj];
#pragma unroll
        for (int t = 0; t < NB; ++t)
          if (t < jj) a -= xr[t] * D[jj][t];
        xr[jj] = a / D[jj][jj];
      }
    }
#pragma unroll
    for (int jj = 0; jj < NB; ++jj)
      if (jj < nbj) crow[jj] = xr[jj];
  }
}

// Trailing update after the panel at column j0: C[i][j] -= sum_k C[i][j0 + k] C[j][j0 + k] on the lower triangle
// beyond the panel.  blockIdx.y selects the matrix, blockIdx.x a pair (ti >= tj) of 64-row tiles.
__global__ void __launch_bounds__(256) chol_trailing_kernel(const CholProblem* probs, int j0) {
  constexpr int NB = kCholNB;
  __shared__ double As[NB][64 + 1];
  __shared__ double Bs[NB][64 + 1];
  const CholProblem p = probs[blockIdx.y];
  const int L = p.L, base = j0 + NB;
  if (base >= L) return;
  const int nt = (L - base + 63) / 64;
  int ti = static_cast<int>((sqrtf(8.f * blockIdx.x + 1.f) - 1.f) * 0.5f);
  while ((ti + 1) * (ti + 2) / 2 <= static_cast<int>(blockIdx.x)) ++ti;
  while (ti * (ti + 1) / 2 > static_cast<int>(blockIdx.x)) --ti;
  const int tj = blockIdx.x - ti * (ti + 1) / 2;
  if (ti >= nt) return;
  const int i0 = base + ti * 64, c0 = base + tj * 64;
  const int t = threadIdx.x;
  for (int x = t; x < NB * 64; x += 256) {
    const int r = x / NB, k = x % NB;  // k contiguous in memory
    As[k][r] = (i0 + r < L) ? p.C[static_cast<long long>(i0 + r) * L + j0 + k] : 0.0;
    Bs[k][r] = (c0 + r < L) ? p.C[static_cast<long long>(c0 + r) * L + j0 + k] : 0.0;
  }
  __syncthreads();
  const int tx = t & 15, ty = t >> 4;
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
#pragma unroll 8
  for (int k = 0; k < NB; ++k) {
    double a[4], b[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) { a[x] = As[k][ty * 4 + x]; b[x] = Bs[k][tx * 4 + x]; }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) acc[x][y] += a[x] * b[y];
  }
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int i = i0 + ty * 4 + x;
    if (i >= L) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int j = c0 + tx * 4 + y;
      if (j <= i) p.C[static_cast<long long>(i) * L + j] -= acc[x][y];
    }
  }
}

// Factor n matrices (the largest of size Lmax).  Panels of 32 columns: the panel step runs one CTA per matrix, the
// trailing update spreads over the whole GPU; 2 Lmax / 32 launches.
inline cudaError_t chol_batched_launch(CholProblem* d_probs, int n, int Lmax, cudaStream_t stream, int64_t* launches) {
  chol_begin_kernel<<<n, 32, 0, stream>>>(d_probs);
  *launches += 1;
  for (int j0 = 0; j0 < Lmax; j0 += kCholNB) {
    chol_panel_kernel<<<n, 256, 0, stream>>>(d_probs, j0);
    *launches += 1;
    const int rows = Lmax - j0 - kCholNB;
    if (rows > 0) {
      const int nt = (rows + 63) / 64;
      chol_trailing_kernel<<<dim3(nt * (nt + 1) / 2, n), 256, 0, stream>>>(d_probs, j0);
      *launches += 1;
    }
  }
  return cudaGetLastError();
}

// The same factorisation with one CTA per matrix and no launches between the panels: for a batch of about as many
// matrices as there are SMs this keeps every SM busy from the first panel to the last, where the launch-per-panel
// version spends most of its time between kernels (a 512 x 512 factor is 16 panels, i.e. 32 launches of a few
// tens of microseconds each, for 45 million multiply-adds).  Per panel: one warp factors the diagonal block in
// registers, every thread solves one row of the panel against it (keeping the solved panel in shared memory,
// column-major), and all threads update the trailing triangle in 4 x 4 register tiles straight in global memory
// (the matrix stays in L2).  Shared memory: 32 x (L - 32) doubles for the panel.
constexpr int kCholCtaThreads = 512;

// Row length of the panel in shared memory: a multiple of 16 bytes, so that four consecutive rows load at once.
template <typename T>
__host__ __device__ inline int chol_cta_ldp(int trailing) {
  return sizeof(T) == 8 ? trailing + 4 - (trailing & 1) : (trailing + 7) & ~3;
}

template <typename T>
inline size_t chol_cta_smem_bytes(int Lmax) {
  const int rows = Lmax > kCholNB ? Lmax - kCholNB : 0;
  return sizeof(T) * static_cast<size_t>(kCholNB) * (chol_cta_ldp<T>(rows) + 4);
}

__device__ __forceinline__ void chol_load4(const double* p, double (&a)[4]) {
  const double2 lo = *reinterpret_cast<const double2*>(p), hi = *reinterpret_cast<const double2*>(p + 2);
  a[0] = lo.x; a[1] = lo.y; a[2] = hi.x; a[3] = hi.y;
}
__device__ __forceinline__ void chol_load4(const float* p, float (&a)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  a[0] = v.x; a[1] = v.y; a[2] = v.z; a[3] = v.w;
}

// The diagonal block of a panel, by one warp: D (nbj x nbj, zero beyond) is replaced by its lower Cholesky factor
// and rdiag receives the reciprocals of the factor's diagonal (zero beyond the block).  Lane i holds row i in
// registers: step k takes the pivot from lane k, scales column k, and every lane subtracts its share of the
// rank-one update with one shuffle per entry.  A function of its own so that its 32 row entries get registers
// whatever the caller needs elsewhere.
template <typename T>
__device__ __noinline__ void chol_diag_block(T (*D)[kCholNB + 1], T* rdiag, int nbj, T tiny, int lane) {
  constexpr int NB = kCholNB;
  T r[NB];
#pragma unroll
  for (int j = 0; j < NB; ++j) r[j] = D[lane][j];
#pragma unroll
  for (int k = 0; k < NB; ++k) {
    T dkk = __shfl_sync(0xffffffffu, r[k], k);
    if (!(dkk > tiny)) dkk = tiny;
    const T lkk = sqrt(dkk);
    const T inv = T(1) / lkk;
    if (lane == k) {
      r[k] = lkk;
      rdiag[k] = k < nbj ? inv : T(0);
    }
    if (lane > k) r[k] = r[k] * inv;
    const T lik = r[k];
#pragma unroll
    for (int j = k + 1; j < NB; ++j) {
      const T ljk = __shfl_sync(0xffffffffu, r[k], j);
      if (lane >= j) r[j] -= lik * ljk;
    }
  }
#pragma unroll
  for (int j = 0; j < NB; ++j) D[lane][j] = (j <= lane && lane < nbj && j < nbj) ? r[j] : T(0);
}

// One row of the panel, held as entries p[jj * ldp] (jj = 0 .. 31) of the k-major panel in shared memory:
// x D^T = c by forward substitution in place.  As soon as x_t is known every later entry takes its share of it, so
// the dependent chain is one multiply and one multiply-add per t.
template <typename T>
__device__ __noinline__ void chol_panel_row(T* p, int ldp, const T (*D)[kCholNB + 1], const T* rdiag) {
  constexpr int NB = kCholNB;
  T a[NB];
#pragma unroll
  for (int jj = 0; jj < NB; ++jj) a[jj] = p[jj * ldp];
#pragma unroll
  for (int t = 0; t < NB; ++t) {
    const T xt = a[t] * rdiag[t];
    a[t] = xt;
#pragma unroll
    for (int jj = t + 1; jj < NB; ++jj) a[jj] -= xt * D[jj][t];
    if ((t & 3) == 3) asm volatile("" ::: "memory");   // keeps the 496 loads of D from being lifted to the front
  }
#pragma unroll
  for (int jj = 0; jj < NB; ++jj) p[jj * ldp] = a[jj];
}

// T = double: the factorisation as described.  T = float: the same on a matrix stored as L x L floats at the same
// address (CholProblem::C reinterpreted); enough for the orthonormalisations between the products of the subspace
// iteration, whose Gram matrices come from the tensor cores with 2^-17 of relative accuracy and carry a shift of
// about 1e-2 on a unit diagonal, and about twice as fast (half the shared-memory traffic per multiply-add, twice
// the arithmetic rate).
template <typename T>
__global__ void __launch_bounds__(kCholCtaThreads, 1) chol_cta_kernel(const CholProblem* probs) {
  constexpr int NB = kCholNB;
  extern __shared__ __align__(16) unsigned char chol_ps_raw[];
  T* chol_ps = reinterpret_cast<T*>(chol_ps_raw);    // panel, k-major: chol_ps[k * ldp + (row - base)]
  __shared__ T D[NB][NB + 1];      // the diagonal block, then its lower Cholesky factor
  __shared__ T rdiag[NB];          // reciprocals of the factor's diagonal
  __shared__ T s_tiny;
  const CholProblem p = probs[blockIdx.x];
  T* C = reinterpret_cast<T*>(p.C);
  const int L = p.L;
  const int tid = threadIdx.x;
  // pivot floor from the diagonal (a pivot that is not above it is replaced by it, see chol_begin_kernel)
  if (tid < 32) {
    T md = 0;
    for (int i = tid; i < L; i += 32) {
      const T v = C[static_cast<long long>(i) * L + i];
      md = v > md ? v : md;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const T v = __shfl_xor_sync(0xffffffffu, md, o);
      md = v > md ? v : md;
    }
    if (tid == 0) s_tiny = sizeof(T) == 8 ? static_cast<T>(fmax(static_cast<double>(md) * 1e-28, 1e-300))
                                          : static_cast<T>(fmax(static_cast<double>(md) * 1e-12, 1e-30));
  }
  __syncthreads();
  const T tiny = s_tiny;
  for (int j0 = 0; j0 < L; j0 += NB) {
    const int nbj = (L - j0 < NB) ? (L - j0) : NB;
    const int base = j0 + nbj;            // first row / column of the trailing part
    const int Tn = L - base;              // its size
    const int ldp = chol_cta_ldp<T>(Tn);
    for (int x = tid; x < NB * NB; x += kCholCtaThreads) {
      const int a = x / NB, b = x % NB;
      D[a][b] = (a < nbj && b < nbj) ? C[static_cast<long long>(j0 + a) * L + j0 + b] : T(0);
    }
    __syncthreads();
    if (tid < 32) chol_diag_block<T>(D, rdiag, nbj, tiny, tid);
    __syncthreads();
    for (int x = tid; x < NB * NB; x += kCholCtaThreads) {
      const int a = x / NB, b = x % NB;
      if (a < nbj && b <= a) C[static_cast<long long>(j0 + a) * L + j0 + b] = D[a][b];
    }
    // panel rows: x D^T = c.  The rows come in through shared memory (a warp reads one row of 32
    // entries at a time, so that global memory sees whole lines), one thread per row then works in place on its
    // column of the k-major panel, and the solved rows go out the same way.
    {
      const int warp = tid >> 5, lane = tid & 31;
      for (int r = warp; r < Tn; r += kCholCtaThreads / 32)
        chol_ps[lane * ldp + r] = (lane < nbj) ? C[static_cast<long long>(base + r) * L + j0 + lane] : T(0);
      __syncthreads();
      for (int r = tid; r < Tn; r += kCholCtaThreads) chol_panel_row<T>(chol_ps + r, ldp, D, rdiag);
      __syncthreads();
      for (int r = warp; r < Tn; r += kCholCtaThreads / 32)
        if (lane < nbj) C[static_cast<long long>(base + r) * L + j0 + lane] = chol_ps[lane * ldp + r];
    }
    __syncthreads();
    // trailing update on the lower triangle: C[i][j] -= sum_k panel[i][k] panel[j][k], 4 x 4 tiles
    if (Tn > 0) {
      const int nt = (Tn + 3) >> 2;
      const int ntiles = nt * (nt + 1) / 2;
      for (int t = tid; t < ntiles; t += kCholCtaThreads) {
        int ti = static_cast<int>((sqrtf(8.f * t + 1.f) - 1.f) * 0.5f);
        while ((ti + 1) * (ti + 2) / 2 <= t) ++ti;
        while (ti * (ti + 1) / 2 > t) --ti;
        const int tj = t - ti * (ti + 1) / 2;
        const int i0 = 4 * ti, c0 = 4 * tj;        // relative to base
        T acc[4][4];
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
          for (int y = 0; y < 4; ++y) acc[x][y] = T(0);
#pragma unroll 4
        for (int k = 0; k < NB; ++k) {
          const T* pk = chol_ps + k * ldp;
          // (rows beyond the trailing part inside the last tile read the padding or the next column's start: finite
          // values that the bounds check below keeps from being stored)
          T a[4], b[4];
          chol_load4(pk + i0, a);
          chol_load4(pk + c0, b);
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) acc[x][y] += a[x] * b[y];
        }
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const int i = base + i0 + x;
          if (i >= L) continue;
#pragma unroll
          for (int y = 0; y < 4; ++y) {
            const int j = base + c0 + y;
            if (j <= i) C[static_cast<long long>(i) * L + j] -= acc[x][y];
          }
        }
      }
    }
    __syncthreads();
  }
}

// Factor n matrices, one CTA each (the list should start with the largest matrices: CTAs are handed out in order).
template <typename T>
inline cudaError_t chol_cta_launch(const CholProblem* d_probs, int n, int Lmax, cudaStream_t stream, int64_t* launches) {
  chol_cta_kernel<T><<<n, kCholCtaThreads, chol_cta_smem_bytes<T>(Lmax), stream>>>(d_probs);
  *launches += 1;
  return cudaGetLastError();
}

// ---------------------------------------------------------------- Q = Y Lf^-T (rows are independent)

// One CTA owns 32 rows of Y (rows x L, fp32) and produces the same rows of Q (fp32) with
// Q Lf^T = Y, Lf the lower Cholesky factor of Y^T Y (fp64).  Column blocks of 32 are solved in
// order; finished columns of Q stay in shared memory (fp64).
struct OrthApply {
  const float* Y;
  float* Q;
  const double* Lf;
  int rows, L;
};

inline size_t orth_apply_smem_bytes(int L) {
  return (static_cast<size_t>(32) * L + 32 * 33) * sizeof(double);
}

__global__ void __launch_bounds__(256) orth_apply_kernel(OrthApply p) {
  constexpr int NB = 32, RB = 32;
  extern __shared__ __align__(16) unsigned char orth_smem_raw[];
  double* Qs = reinterpret_cast<double*>(orth_smem_raw);  // RB x L (finished columns)
  double* Ls = Qs + static_cast<size_t>(RB) * p.L;        // NB x (NB + 1) chunk of Lf
  const int tid = threadIdx.x;
  const int r0 = blockIdx.x * RB;
  const int L = p.L;
  const int row = tid >> 3;      // 0..31
  const int cg = (tid & 7) * 4;  // 4 columns of the current block
  for (int j0 = 0; j0 < L; j0 += NB) {
    const int nbj = (L - j0 < NB) ? (L - j0) : NB;
    double acc[4];
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int col = j0 + cg + y;
      acc[y] = (r0 + row < p.rows && col < L)
                   ? static_cast<double>(p.Y[static_cast<long long>(r0 + row) * L + col])
                   : 0.0;
    }
    for (int k0 = 0; k0 < j0; k0 += NB) {
      __syncthreads();
      for (int x = tid; x < NB * NB; x += 256) {
        const int a = x / NB, b = x % NB;
        Ls[a * (NB + 1) + b] = (a < nbj) ? p.Lf[static_cast<long long>(j0 + a) * L + k0 + b] : 0.0;
      }
      __syncthreads();
#pragma unroll 8
      for (int b = 0; b < NB; ++b) {
        const double qv = Qs[static_cast<size_t>(row) * L + k0 + b];
        acc[0] -= qv * Ls[(cg + 0) * (NB + 1) + b];
        acc[1] -= qv * Ls[(cg + 1) * (NB + 1) + b];
        acc[2] -= qv * Ls[(cg + 2) * (NB + 1) + b];
        acc[3] -= qv * Ls[(cg + 3) * (NB + 1) + b];
      }
    }
    __syncthreads();
#pragma unroll
    for (int y = 0; y < 4; ++y)
      if (cg + y < nbj) Qs[static_cast<size_t>(row) * L + j0 + cg + y] = acc[y];
    for (int x = tid; x < NB * NB; x += 256) {
      const int a = x / NB, b = x % NB;
      Ls[a * (NB + 1) + b] = (a < nbj && b < nbj) ? p.Lf[static_cast<long long>(j0 + a) * L + j0 + b] : 0.0;
    }
    __syncthreads();
    if (tid < RB) {
      double* q = Qs + static_cast<size_t>(tid) * L + j0;
      for (int jj = 0; jj < nbj; ++jj) {
        double a = q[jj];
        for (int t = 0; t < jj; ++t) a -= q[t] * Ls[jj * (NB + 1) + t];
        q[jj] = a / Ls[jj * (NB + 1) + jj];
      }
    }
    __syncthreads();
  }
  for (int x = tid; x < RB * L; x += 256) {
    const int a = x / L, b = x % L;
    if (r0 + a < p.rows)
      p.Q[static_cast<long long>(r0 + a) * L + b] = static_cast<float>(Qs[static_cast<size_t>(a) * L + b]);
  }
}

// ---------------------------------------------------------------- working copies of P

// Working copies of a projector P32 (rows x rp): P16 (rows x ldp) and its transpose Pt16 (rp x ldpt), both
// holding the bf16-rounded values.  One of the two is stored as bf16 and the other as fp16 (p16_is_half says
// which): a bf16 number converts to fp16 without error unless it is below 2^-17 in magnitude, where the error is
// at most 2^-25, far below the resolution of an orthonormal column's entries.
// Block (32, 8).
__device__ __forceinline__ uint16_t working_bits(float val, bool as_half) {
  const __nv_bfloat16 b = __float2bfloat16_rn(val);
  if (!as_half) return __bfloat16_as_ushort(b);
  return __half_as_ushort(__float2half_rn(__bfloat162float(b)));
}

__global__ void working_copies_kernel(const float* P32, uint16_t* P16, uint16_t* Pt16, int rows, int rp, int ldp,
                                      int ldpt, int p16_is_half) {
  __shared__ float tile[32][33];
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  for (int a = threadIdx.y; a < 32; a += blockDim.y) {
    const int i = i0 + a, j = j0 + threadIdx.x;
    float val = 0.f;
    if (i < rows && j < rp) {
      val = P32[static_cast<long long>(i) * rp + j];
      P16[static_cast<long long>(i) * ldp + j] = working_bits(val, p16_is_half != 0);
    }
    tile[a][threadIdx.x] = val;
  }
  __syncthreads();
  for (int a = threadIdx.y; a < 32; a += blockDim.y) {
    const int j = j0 + a, i = i0 + threadIdx.x;
    if (i < rows && j < rp) Pt16[static_cast<long long>(j) * ldpt + i] = working_bits(tile[threadIdx.x][a], p16_is_half == 0);
  }
}

// The same for a list of matrices in one launch, reading the new basis where the refresh left it (src) and writing
// the fp32 master as well.  CTA t works on a 32 x 32 tile; tile_start[j] is the first tile of job j (n_jobs + 1
// entries, ascending).
struct WorkingJob {
  const float* src;   // rows x rp, dense
  float* P32;
  uint16_t* P16;
  uint16_t* Pt16;
  int rows, rp, ldp, ldpt;
  int p16_is_half;
  int tiles_x;        // tiles along the rp columns
};

__global__ void working_copies_grouped_kernel(const WorkingJob* jobs, const int* tile_start, int n_jobs) {
  __shared__ float tile[32][33];
  int lo = 0, hi = n_jobs;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (tile_start[mid] <= static_cast<int>(blockIdx.x)) lo = mid; else hi = mid;
  }
  const WorkingJob jb = jobs[lo];
  const int t = static_cast<int>(blockIdx.x) - tile_start[lo];
  const int i0 = (t / jb.tiles_x) * 32, j0 = (t % jb.tiles_x) * 32;
  for (int a = threadIdx.y; a < 32; a += blockDim.y) {
    const int i = i0 + a, j = j0 + threadIdx.x;
    float val = 0.f;
    if (i < jb.rows && j < jb.rp) {
      val = jb.src[static_cast<long long>(i) * jb.rp + j];
      jb.P32[static_cast<long long>(i) * jb.rp + j] = val;
      jb.P16[static_cast<long long>(i) * jb.ldp + j] = working_bits(val, jb.p16_is_half != 0);
    }
    tile[a][threadIdx.x] = val;
  }
  __syncthreads();
  for (int a = threadIdx.y; a < 32; a += blockDim.y) {
    const int j = j0 + a, i = i0 + threadIdx.x;
    if (i < jb.rows && j < jb.rp) jb.Pt16[static_cast<long long>(j) * jb.ldpt + i] = working_bits(tile[threadIdx.x][a], jb.p16_is_half == 0);
  }
}

// A refreshed basis that is no basis: all zeros (the gradient of a frozen layer: every product of the iteration is
// zero and nothing can be normalised) or with entries that are not finite (a gradient with such entries).  Any
// orthonormal basis serves a zero gradient, so such a matrix gets the first r' unit vectors; the second case also
// raises the matrix's status word.  Two launches over a list of matrices: sums, then the repair.
struct BasisJob {
  float* Ya;       // rows x rp, dense: the basis, in one of the two buffers of the refresh
  float* Yb;
  double* acc;     // [0]: sum of squares, [1]: number of entries that are not finite (cleared by the caller)
  int* status;
  int rows, rp;
};

__global__ void __launch_bounds__(256) basis_check_kernel(const BasisJob* jobs, int in_a) {
  __shared__ double red[8];
  __shared__ int bad_any;
  const BasisJob jb = jobs[blockIdx.y];
  const float* Y = in_a ? jb.Ya : jb.Yb;
  const long long n = static_cast<long long>(jb.rows) * jb.rp;
  if (threadIdx.x == 0) bad_any = 0;
  __syncthreads();
  double s = 0.0;
  int bad = 0;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += 256ll * gridDim.x) {
    const float x = Y[i];
    if (isfinite(x)) s += static_cast<double>(x) * static_cast<double>(x);
    else bad = 1;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  if (bad) bad_any = 1;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += red[w];
    if (t != 0.0) atomicAdd(jb.acc, t);
    if (bad_any) atomicAdd(jb.acc + 1, 1.0);
  }
}

__global__ void __launch_bounds__(256) basis_repair_kernel(const BasisJob* jobs, int in_a) {
  const BasisJob jb = jobs[blockIdx.y];
  const bool nonfinite = jb.acc[1] > 0.0;
  if (!nonfinite && jb.acc[0] > 0.0) return;
  float* Y = in_a ? jb.Ya : jb.Yb;
  const long long n = static_cast<long long>(jb.rows) * jb.rp;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += 256ll * gridDim.x)
    Y[i] = (i / jb.rp == i % jb.rp) ? 1.f : 0.f;
  if (nonfinite && blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(jb.status, 0, 7 /* NGALORE_ERR_NONFINITE */);
}

// dst (rows x cols, dense fp32) = src (rows x cols, leading dimension ld; fp16 or bf16 bits)
__global__ void widen_16_kernel(const uint16_t* src, float* dst, long long n, int cols, int ld, int is_half) {
  const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  if (i >= n) return;
  const uint16_t bits = src[(i / cols) * ld + (i % cols)];
  dst[i] = is_half ? __half2float(__ushort_as_half(bits)) : __bfloat162float(__ushort_as_bfloat16(bits));
}

// dst (cols x ld_dst, bf16, padding columns left untouched) = src^T for src (rows x cols, bf16).  Block (32, 8).
__global__ void transpose_bf16_kernel(const uint16_t* src, uint16_t* dst, int rows, int cols, int ld_dst) {
  __shared__ uint16_t tile[32][33];
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  for (int a = threadIdx.y; a < 32; a += blockDim.y) {
    const int i = i0 + a, j = j0 + threadIdx.x;
    tile[a][threadIdx.x] = (i < rows && j < cols) ? src[static_cast<long long>(i) * cols + j] : uint16_t(0);
  }
  __syncthreads();
  for (int a = threadIdx.y; a < 32; a += blockDim.y) {
    const int j = j0 + a, i = i0 + threadIdx.x;
    if (i < rows && j < cols) dst[static_cast<long long>(j) * ld_dst + i] = tile[threadIdx.x][a];
  }
}

}  // namespace ngalore
