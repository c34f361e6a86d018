// Rayleigh-Ritz rotation of the subspace refresh (Sec. 1: P holds the left singular VECTORS of the gradient,
// not just a basis of their span; Sec. 2.2 runs Adam element by element in the coordinates P defines, so the
// basis inside the subspace matters wherever the singular values are separated).
//
// Given an orthonormal basis Q of the subspace found by the subspace iteration, the Ritz vectors are P = Q V with
// V the eigenvectors of C = (Q^T G)(Q^T G)^T = Z^T Z, Z = G^T Q.  This file diagonalises the small symmetric
// matrices C (L x L, L = r' <= 875, one per weight matrix, all in one batch) by a one-sided block Jacobi method:
// the columns of a working matrix X (started as C, scaled to a unit largest diagonal entry) are rotated against
// each other until they are mutually orthogonal; the accumulated rotation is V and the column norms are the
// eigenvalues.  The unit of work is one pair of 16-column blocks of one matrix: a CTA forms the 32 x 32 Gram
// matrix of its 32 columns, four warps diagonalise that by cyclic two-sided Jacobi rotations, and a CTA applies the
// resulting 32 x 32 rotation to the 32 columns of X and of V.  The block pairs of a round are disjoint
// (round-robin ordering), so a round is a few launches over every matrix; a sweep is (blocks - 1) rounds.
//
// The rotation can be limited to the span of the leading k columns of the basis (JacobiMat::L = k < basis width):
// the matrix diagonalised is then the leading k x k block of C, the first k columns of P become the Ritz vectors
// of G within the span of the first k basis vectors, and the remaining basis vectors stay as they are.  The
// subspace iteration orders its basis by strength (every orthonormalisation works through the columns in order),
// so what the leading Ritz vectors lose is the part of the dominant directions that sits in the later columns,
// which is at the rounding level of the iteration.  That is the default for wide bases, because the cost grows with
// the square of the number of blocks: a singular vector is only determined where its singular value is separated
// from its neighbours, at most about a hundred values can be separated by 1e-2 sigma_1 from both neighbours, and
// for decaying spectra those sit at the front.
//
// The working matrix X is single precision: it only decides the rotation angles, and the Ritz vectors of
// gap-separated values come out to about 1e-6 / relative gap.  V is kept in double precision and every 32 x 32
// rotation is re-orthogonalised (one Newton-Schulz step in double precision) before it is applied, so that V, a
// product of a few hundred of them, is orthogonal to rounding instead of to 1e-4.  That matters for gradients
// whose singular values span a factor of a few thousand: P = Q V inherits what V lacks in orthogonality, any later
// orthonormalisation of P moves a column by the amount it finds it non-orthogonal to the columns before it, and
// 1e-4 of the strongest singular directions mixed into the weak ones is as much as the weak directions carry
// themselves.  With V orthogonal and Q orthonormal, P = Q V needs no further orthonormalisation.
#pragma once

#include "common.cuh"

namespace ngalore {

constexpr int kJacBlock = 16;           // columns per block; a CTA rotates two blocks against each other
constexpr int kJacCols = 2 * kJacBlock;
constexpr int kJacThreads = 256;
constexpr int kJacMaxSweeps = 12;
constexpr float kJacTol = 1e-5f;        // a pair of columns counts as orthogonal below this cosine
constexpr int kJacInnerSweeps = 2;      // sweeps over the 32 x 32 Gram matrix of a block pair per visit

struct JacobiMat {
  float* XT;    // L x ld: row i is column i of the working matrix X
  double* VT;   // L x ld: row i is column i of the accumulated rotation V (may share the memory of the fp64 input
                // of jacobi_init_kernel: that kernel reads all of its input before it writes V)
  int L, ld;    // ld >= L, a multiple of 4
  int nblk;     // number of 16-column blocks, rounded up to an even number (>= 2)
  int* flags;   // [0]: some pair was rotated in the sweep in progress; [1]: converged, nothing left to do
};

// Circle method: round r of a tournament of n players (n even), table l (0 .. n/2 - 1).
__device__ __forceinline__ void round_robin_pair(int n, int r, int l, int& a, int& b) {
  if (l == 0) {
    a = n - 1;
    b = r % (n - 1);
  } else {
    a = (r + l) % (n - 1);
    b = (r - l + 2 * (n - 1)) % (n - 1);
  }
}

// X = (S + S^T) / (2 max_i S_ii) from a symmetric matrix given in fp32 (S32, leading dimension lds) or fp64
// (S64); V = I; flags cleared.  One CTA per matrix.
struct JacobiInit {
  const float* S32;
  const double* S64;
  int lds;
};

__global__ void __launch_bounds__(256) jacobi_init_kernel(const JacobiMat* mats, const JacobiInit* inits) {
  __shared__ float red[8];
  const JacobiMat m = mats[blockIdx.x];
  const JacobiInit in = inits[blockIdx.x];
  float md = 0.f;
  for (int i = threadIdx.x; i < m.L; i += 256) {
    const long long d = static_cast<long long>(i) * in.lds + i;
    md = fmaxf(md, in.S32 != nullptr ? in.S32[d] : static_cast<float>(in.S64[d]));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) md = fmaxf(md, __shfl_xor_sync(0xffffffffu, md, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = md;
  __syncthreads();
  md = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) md = fmaxf(md, red[w]);
  const double inv = md > 0.f ? 0.5 / static_cast<double>(md) : 0.0;
  const long long total = static_cast<long long>(m.L) * m.ld;
  for (long long x = threadIdx.x; x < total; x += 256) {
    const int i = static_cast<int>(x / m.ld), j = static_cast<int>(x % m.ld);
    float xv = 0.f;
    if (j < m.L) {
      const long long a = static_cast<long long>(i) * in.lds + j, b = static_cast<long long>(j) * in.lds + i;
      const double s = in.S32 != nullptr ? static_cast<double>(in.S32[a]) + static_cast<double>(in.S32[b])
                                         : in.S64[a] + in.S64[b];
      xv = static_cast<float>(s * inv);
    }
    m.XT[x] = xv;
  }
  __syncthreads();  // V may overwrite the input
  for (long long x = threadIdx.x; x < total; x += 256) m.VT[x] = (x / m.ld == x % m.ld) ? 1.0 : 0.0;
  if (threadIdx.x < 2) m.flags[threadIdx.x] = 0;
}

inline size_t jacobi_smem_bytes(int ld_max) {
  return static_cast<size_t>(kJacCols) * (ld_max + 4) * sizeof(float);
}

// Scratch of one block pair of the round in progress: its Gram matrix, the rotation found for it, and whether
// there is anything to rotate.
struct JacobiSlot {
  float A[kJacCols][kJacCols];
  float J[kJacCols][kJacCols];    // J[a][b] = rotation entry (b, a): new column a = sum_b J[a][b] * old column b
  double Jd[kJacCols][kJacCols];  // the same, re-orthogonalised in double precision
  int active;
  int pad[3];
};

struct JacobiPairInfo {
  int bi, bj;
  bool live;
};

__device__ __forceinline__ JacobiPairInfo jacobi_pair_of(const JacobiMat& m, int round, int table) {
  JacobiPairInfo pi{0, 0, false};
  if (table >= m.nblk / 2) return pi;
  if (*reinterpret_cast<volatile int*>(m.flags + 1)) return pi;
  round_robin_pair(m.nblk, round % (m.nblk - 1), table, pi.bi, pi.bj);
  // (a block beyond L is padding: its columns load as zeros and never rotate; the columns of its partner are
  // still rotated against each other, which is all there is to do when the matrix has a single block)
  pi.live = !(pi.bi * kJacBlock >= m.L && pi.bj * kJacBlock >= m.L);
  return pi;
}

// Step 1 of a round: Gram matrix of the 32 columns of every block pair.  blockIdx.y = matrix, blockIdx.x = table
// of the round-robin round; slot = blockIdx.y * gridDim.x + blockIdx.x.
__global__ void __launch_bounds__(kJacThreads) jacobi_gram_kernel(const JacobiMat* mats, JacobiSlot* slots, int round) {
  extern __shared__ __align__(16) float jac_xs[];               // 32 rows x (ld + 4)
  __shared__ float Ap[4][kJacCols][kJacCols + 1];               // one partial Gram matrix per group of threads
  __shared__ int s_any;
  const JacobiMat m = mats[blockIdx.y];
  JacobiSlot& slot = slots[blockIdx.y * gridDim.x + blockIdx.x];
  const JacobiPairInfo pi = jacobi_pair_of(m, round, blockIdx.x);
  const int tid = threadIdx.x;
  if (!pi.live) {
    if (tid == 0) slot.active = 0;
    return;
  }
  const int L = m.L, ld = m.ld, lds = ld + 4;
  const int quads = ld >> 2;
  for (int a = tid >> 5; a < kJacCols; a += kJacThreads / 32) {       // a warp per row: coalesced, no divisions
    const int gr = (a < kJacBlock ? pi.bi : pi.bj) * kJacBlock + (a & (kJacBlock - 1));
    for (int q = tid & 31; q < quads; q += 32) {
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (gr < L) v = *reinterpret_cast<const float4*>(m.XT + static_cast<long long>(gr) * ld + 4 * q);
      *reinterpret_cast<float4*>(jac_xs + a * lds + 4 * q) = v;
    }
  }
  if (tid == 0) s_any = 0;
  __syncthreads();
  // 64 tiles of 4 x 4 entries; four groups of threads share the length of the columns
  {
    const int kg = tid >> 6, tile = tid & 63, ta = tile >> 3, tb = tile & 7;
    const float* ra = jac_xs + (4 * ta) * lds;
    const float* rb = jac_xs + (4 * tb) * lds;
    float g[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) g[x][y] = 0.f;
    for (int q = kg; q < quads; q += 4) {
      float4 a[4], b[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        a[x] = *reinterpret_cast<const float4*>(ra + x * lds + 4 * q);
        b[x] = *reinterpret_cast<const float4*>(rb + x * lds + 4 * q);
      }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y)
          g[x][y] += a[x].x * b[y].x + a[x].y * b[y].y + a[x].z * b[y].z + a[x].w * b[y].w;
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) Ap[kg][4 * ta + x][4 * tb + y] = g[x][y];
  }
  __syncthreads();
  // add the four partial matrices in a fixed order (entry (p, q) and entry (q, p) then agree to the bit); is any
  // pair of columns further from orthogonal than the tolerance?
  auto entry = [&](int p, int q) { return (Ap[0][p][q] + Ap[1][p][q]) + (Ap[2][p][q] + Ap[3][p][q]); };
  int any = 0;
  for (int x = tid; x < kJacCols * kJacCols; x += kJacThreads) {
    const int p = x / kJacCols, q = x % kJacCols;
    const float v = p <= q ? entry(p, q) : entry(q, p);
    slot.A[p][q] = v;
    if (p < q && v * v > kJacTol * kJacTol * entry(p, p) * entry(q, q)) any = 1;
  }
  if (any) atomicOr(&s_any, 1);
  __syncthreads();
  if (tid == 0) {
    slot.active = s_any;
    if (s_any) atomicOr(m.flags, 1);
  }
}

// Step 2: one CTA of four warps per block pair diagonalises its Gram matrix by cyclic two-sided Jacobi rotations, 16
// disjoint ones per step: A <- R^T A R, J <- J R.  With partner(j) the column that column j is paired with in a
// step, column j of A R is ca[j] * column j + cb[j] * column partner(j); rows likewise.  Sixteen threads find the
// angles; then every thread (row r, eight columns) forms its entries of B = A R, and after a barrier its entries of
// R^T B and of J R.  A solve is a chain of dependent steps, so its latency is what a round of the rotation costs:
// four warps per solve instead of one cut it about fivefold.  A few sweeps are enough: the outer iteration comes
// back to every pair.
constexpr int kJacInnerThreads = 128;

__global__ void __launch_bounds__(kJacInnerThreads) jacobi_inner_kernel(JacobiSlot* slots, int n_slots) {
  __shared__ float As[kJacCols][kJacCols + 1];
  __shared__ float Bs[kJacCols][kJacCols + 1];
  __shared__ float JT[kJacCols][kJacCols + 1];   // JT[a][b] = J[b][a]
  __shared__ float ca[kJacCols], cb[kJacCols];
  __shared__ unsigned char partner[kJacCols];
  JacobiSlot& slot = slots[blockIdx.x];
  if (slot.active == 0) return;
  const int tid = threadIdx.x;
  const int r = tid >> 2, j0 = (tid & 3) * 8;     // this thread: row r, columns j0 .. j0 + 7
#pragma unroll
  for (int y = 0; y < 8; ++y) {
    As[r][j0 + y] = slot.A[r][j0 + y];
    JT[r][j0 + y] = (r == j0 + y) ? 1.f : 0.f;
  }
  __syncthreads();
  for (int sweep = 0; sweep < kJacInnerSweeps; ++sweep) {
    int rotated = 0;
    for (int step = 0; step < kJacCols - 1; ++step) {
      if (tid < kJacBlock) {
        int p, q;
        round_robin_pair(kJacCols, step, tid, p, q);
        const float app = As[p][p], aqq = As[q][q], apq = As[p][q];
        float c = 1.f, sn = 0.f;
        if (apq * apq > 1e-12f * app * aqq && apq != 0.f) {
          const float tau = (aqq - app) / (2.f * apq);
          const float t = (tau >= 0.f ? 1.f : -1.f) / (fabsf(tau) + sqrtf(1.f + tau * tau));
          c = rsqrtf(1.f + t * t);
          sn = t * c;
          rotated = 1;
        }
        ca[p] = c; cb[p] = -sn; partner[p] = static_cast<unsigned char>(q);
        ca[q] = c; cb[q] = sn; partner[q] = static_cast<unsigned char>(p);
      }
      __syncthreads();
      float t[8];
#pragma unroll
      for (int y = 0; y < 8; ++y) t[y] = ca[j0 + y] * As[r][j0 + y] + cb[j0 + y] * As[r][partner[j0 + y]];
#pragma unroll
      for (int y = 0; y < 8; ++y) Bs[r][j0 + y] = t[y];                            // B = A R
      __syncthreads();
      const float car = ca[r], cbr = cb[r];
      const int pr = partner[r];
#pragma unroll
      for (int y = 0; y < 8; ++y) {
        As[r][j0 + y] = car * Bs[r][j0 + y] + cbr * Bs[pr][j0 + y];                // A <- R^T B
        t[y] = car * JT[r][j0 + y] + cbr * JT[pr][j0 + y];                         // row r of JT = column r of J
      }
      __syncthreads();
#pragma unroll
      for (int y = 0; y < 8; ++y) JT[r][j0 + y] = t[y];
    }
    if (!__syncthreads_or(rotated)) break;
  }
  __syncthreads();
#pragma unroll
  for (int y = 0; y < 8; ++y) slot.J[r][j0 + y] = JT[r][j0 + y];
}

// Step 3: the rotation of every active block pair is made orthogonal to second order, J <- J (I - (J^T J - I) / 2),
// in double precision.  One CTA per slot.
__global__ void __launch_bounds__(kJacThreads) jacobi_polish_kernel(JacobiSlot* slots) {
  __shared__ float JT[kJacCols][kJacCols + 1];   // JT[a][b] = J[b][a] as the inner kernel left it
  __shared__ float Es[kJacCols][kJacCols + 1];   // J^T J - I
  JacobiSlot& slot = slots[blockIdx.x];
  if (slot.active == 0) return;
  const int tid = threadIdx.x;
  for (int x = tid; x < kJacCols * kJacCols; x += kJacThreads) JT[x / kJacCols][x % kJacCols] = slot.J[x / kJacCols][x % kJacCols];
  __syncthreads();
  for (int x = tid; x < kJacCols * kJacCols; x += kJacThreads) {
    const int a = x / kJacCols, b = x % kJacCols;
    double e = (a == b) ? -1.0 : 0.0;
#pragma unroll 8
    for (int k = 0; k < kJacCols; ++k) e += static_cast<double>(JT[a][k]) * static_cast<double>(JT[b][k]);  // (J^T J)_ab
    Es[a][b] = static_cast<float>(e);
  }
  __syncthreads();
  for (int x = tid; x < kJacCols * kJacCols; x += kJacThreads) {
    const int r = x % kJacCols, a = x / kJacCols;
    double v = static_cast<double>(JT[a][r]);                                                              // J[r][a]
#pragma unroll 8
    for (int k = 0; k < kJacCols; ++k) v -= 0.5 * static_cast<double>(JT[k][r]) * static_cast<double>(Es[k][a]);
    slot.Jd[a][r] = v;
  }
}

// Step 4: new column a = sum_b J[a][b] (old column b) for the 32 columns of every active block pair, X in single
// and V in double precision.  blockIdx.z splits the length of the columns.
constexpr int kJacApplyThreads = 128;

__global__ void __launch_bounds__(kJacApplyThreads, 3) jacobi_apply_kernel(const JacobiMat* mats, const JacobiSlot* slots, int round) {
  __shared__ double Jd[kJacCols][kJacCols + 1];
  __shared__ __align__(16) float Jf[kJacCols][kJacCols + 4];
  const JacobiMat m = mats[blockIdx.y];
  const JacobiSlot& slot = slots[blockIdx.y * gridDim.x + blockIdx.x];
  if (slot.active == 0) return;
  int bi, bj;
  round_robin_pair(m.nblk, round % (m.nblk - 1), blockIdx.x, bi, bj);
  const int tid = threadIdx.x;
  const int L = m.L, ld = m.ld;
  auto global_row = [&](int a) { return (a < kJacBlock ? bi : bj) * kJacBlock + (a & (kJacBlock - 1)); };
  for (int x = tid; x < kJacCols * kJacCols; x += kJacApplyThreads) {
    const double v = slot.Jd[x / kJacCols][x % kJacCols];
    Jd[x / kJacCols][x % kJacCols] = v;
    Jf[x / kJacCols][x % kJacCols] = static_cast<float>(v);
  }
  __syncthreads();
  // one element of every column per thread: 32 loads in flight, then 32 x 32 multiply-adds, then 32 stores
  const int k = blockIdx.z * kJacApplyThreads + tid;
  if (k >= ld) return;
  {
    float x[kJacCols];
#pragma unroll
    for (int b = 0; b < kJacCols; ++b) {
      const int gr = global_row(b);
      x[b] = gr < L ? m.XT[static_cast<long long>(gr) * ld + k] : 0.f;
    }
#pragma unroll 4
    for (int a = 0; a < kJacCols; ++a) {
      float acc = 0.f;
#pragma unroll
      for (int b4 = 0; b4 < kJacCols; b4 += 4) {
        const float4 j = *reinterpret_cast<const float4*>(&Jf[a][b4]);
        acc += j.x * x[b4] + j.y * x[b4 + 1] + j.z * x[b4 + 2] + j.w * x[b4 + 3];
      }
      const int gr = global_row(a);
      if (gr < L) m.XT[static_cast<long long>(gr) * ld + k] = acc;
    }
  }
  {
    double v[kJacCols];
#pragma unroll
    for (int b = 0; b < kJacCols; ++b) {
      const int gr = global_row(b);
      v[b] = gr < L ? m.VT[static_cast<long long>(gr) * ld + k] : 0.0;
    }
#pragma unroll 4
    for (int a = 0; a < kJacCols; ++a) {
      double acc = 0.0;
#pragma unroll
      for (int b = 0; b < kJacCols; ++b) acc += Jd[a][b] * v[b];
      const int gr = global_row(a);
      if (gr < L) m.VT[static_cast<long long>(gr) * ld + k] = acc;
    }
  }
}

// End of a sweep: a matrix none of whose pairs was rotated is done.
__global__ void jacobi_sweep_end_kernel(const JacobiMat* mats, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  int* f = mats[i].flags;
  if (f[0] == 0) f[1] = 1;
  f[0] = 0;
}

// Order the Ritz vectors by falling eigenvalue (the norm of a column of X) and write the rotation of the whole
// basis, width W >= L: its leading L x L block is V with its columns in that order, the rest is the identity.  As fp32
// (out32, W x ld32, entry (k, j) = component k of vector j) and / or as two bf16 parts (hi, lo, W x ld16) for the
// tensor-core product Q V.
struct JacobiOut {
  float* out32;
  int ld32;
  __nv_bfloat16 *hi, *lo;
  int ld16;
  int W;
};

constexpr int kJacMaxL = 880;     // largest r' the refresh accepts, rounded up
constexpr int kJacFinishSplit = 8;  // CTAs per matrix in the finish kernel

// blockIdx.x = matrix, blockIdx.y = share of the vectors to write.
__global__ void __launch_bounds__(256) jacobi_finish_kernel(const JacobiMat* mats, const JacobiOut* outs) {
  __shared__ float nrm[kJacMaxL];
  __shared__ int rank_of[kJacMaxL];
  const JacobiMat m = mats[blockIdx.x];
  const JacobiOut o = outs[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = warp; i < m.L; i += 8) {
    float s = 0.f;
    for (int k = lane; k < m.L; k += 32) {
      const float x = m.XT[static_cast<long long>(i) * m.ld + k];
      s += x * x;
    }
#pragma unroll
    for (int of = 16; of > 0; of >>= 1) s += __shfl_xor_sync(0xffffffffu, s, of);
    if (lane == 0) nrm[i] = s;
  }
  __syncthreads();
  // position of column i in the falling order (ties by index); position -> column
  for (int i = threadIdx.x; i < m.L; i += 256) {
    const float mine = nrm[i];
    int pos = 0;
    for (int j = 0; j < m.L; ++j) {
      const float other = nrm[j];
      pos += (other > mine || (other == mine && j < i)) ? 1 : 0;
    }
    rank_of[pos] = i;
  }
  __syncthreads();
  for (int j = blockIdx.y; j < o.W; j += gridDim.y) {  // vector j; reads run along its components
    const double* src = j < m.L ? m.VT + static_cast<long long>(rank_of[j]) * m.ld : nullptr;
    for (int k = threadIdx.x; k < o.W; k += 256) {
      const float v = (j < m.L && k < m.L) ? static_cast<float>(src[k]) : ((j == k) ? 1.f : 0.f);
      if (o.out32 != nullptr) o.out32[static_cast<long long>(k) * o.ld32 + j] = v;
      if (o.hi != nullptr) {
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        o.hi[static_cast<long long>(k) * o.ld16 + j] = h;
        o.lo[static_cast<long long>(k) * o.ld16 + j] = __float2bfloat16_rn(v - __bfloat162float(h));
      }
    }
  }
}

// Diagonalise n matrices (descriptors d_mats, already initialised by jacobi_init_kernel); nblk_max and ld_max are
// the largest block count and leading dimension among them; slots: scratch of n * nblk_max / 2 entries.
inline cudaError_t jacobi_batched_launch(const JacobiMat* d_mats, int n, int nblk_max, int ld_max, JacobiSlot* slots,
                                         cudaStream_t stream, int64_t* launches) {
  const size_t smem = jacobi_smem_bytes(ld_max);
  const int tables = nblk_max / 2, n_slots = n * tables;
  const int parts = (ld_max + kJacApplyThreads - 1) / kJacApplyThreads;
  for (int sweep = 0; sweep < kJacMaxSweeps; ++sweep) {
    for (int round = 0; round < nblk_max - 1; ++round) {
      const int r = sweep * (nblk_max - 1) + round;
      jacobi_gram_kernel<<<dim3(tables, n), kJacThreads, smem, stream>>>(d_mats, slots, r);
      jacobi_inner_kernel<<<n_slots, kJacInnerThreads, 0, stream>>>(slots, n_slots);
      jacobi_polish_kernel<<<n_slots, kJacThreads, 0, stream>>>(slots);
      jacobi_apply_kernel<<<dim3(tables, n, parts), kJacApplyThreads, 0, stream>>>(d_mats, slots, r);
      *launches += 4;
    }
    jacobi_sweep_end_kernel<<<(n + 127) / 128, 128, 0, stream>>>(d_mats, n);
    *launches += 1;
  }
  return cudaGetLastError();
}

inline int jacobi_blocks(int L) {
  int nb = (L + kJacBlock - 1) / kJacBlock;
  if (nb < 2) nb = 2;
  return (nb + 1) & ~1;
}

}  // namespace ngalore
