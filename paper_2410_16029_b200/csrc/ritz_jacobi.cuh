// Rayleigh-Ritz rotation of the subspace refresh (Sec. 1: P holds the left singular VECTORS of the gradient,
// not just a basis of their span; Sec. 2.2 runs Adam element by element in the coordinates P defines, so the
// basis inside the subspace matters wherever the singular values are separated).
//
// Given an orthonormal basis Q of the subspace found by the subspace iteration, the Ritz vectors are P = Q V with
// V the eigenvectors of C = (Q^T G)(Q^T G)^T = Z^T Z, Z = G^T Q.  This file diagonalises the small symmetric
// matrices C (L x L, L = r' <= 875, one per weight matrix, all in one batch) by a one-sided block Jacobi method:
// the columns of a working matrix X (started as C, scaled to a unit largest diagonal entry) are rotated against
// each other until they are mutually orthogonal; the accumulated rotation is V and the column norms are the
// eigenvalues.  The unit of work is one pair of 16-column blocks of one matrix: the 32 x 32 Gram matrix of its 32
// columns is diagonalised by cyclic two-sided Jacobi rotations, and the resulting 32 x 32 rotation is applied to the
// 32 columns of X and of V.  The block pairs of a round are disjoint (round-robin ordering); a sweep is
// (blocks - 1) rounds.  All of it is one launch: a cluster of CTAs per matrix shares the pairs of a round and meets
// at a cluster barrier between rounds (jacobi_cluster_kernel below).
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
constexpr int kJacMaxSweeps = 12;
constexpr float kJacTol = 1e-5f;        // a pair of columns counts as orthogonal below this cosine
constexpr int kJacInnerSweeps = 1;      // sweeps over the 32 x 32 Gram matrix of a block pair per visit

struct JacobiMat {
  float* XT;    // L x ld: row i is column i of the working matrix X
  double* VT;   // L x ld: row i is column i of the accumulated rotation V (may share the memory of the fp64 input
                // of jacobi_init_kernel: that kernel reads all of its input before it writes V)
  int L, ld;    // ld >= L, a multiple of 4
  int nblk;     // number of 16-column blocks, rounded up to an even number (>= 2)
  int* flags;   // kJacMaxSweeps words: [i] != 0 once some pair was rotated in sweep i
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
  if (threadIdx.x < kJacMaxSweeps) m.flags[threadIdx.x] = 0;
}

// One launch diagonalises every matrix: a cluster of kJacCluster CTAs per matrix, each CTA working on two block
// pairs of a round at a time.  The pairs of a round are disjoint, so within a round a CTA reads and writes only the
// columns of its own pairs; between rounds the blocks change partners, and a cluster barrier (release / acquire)
// makes the columns the other CTAs wrote visible.  X and V stay in global memory (they live in L2: a quarter and
// half a megabyte per matrix) and are read past L1.  Per pair: the 32 x 32 Gram matrix of its columns (staged
// through shared memory 64 rows at a time), its eigenvectors by cyclic two-sided Jacobi rotations on 64 threads (both
// pairs of the CTA at once), one Newton-Schulz step in double precision that makes the 32 x 32 rotation orthogonal
// to second order, and the rotation applied to the pair's columns of X (single) and V (double precision).  A sweep
// in which no pair of any round was rotated ends the matrix; all CTAs of a cluster read the same flag after the same
// barrier, so they leave together.
constexpr int kJacCluster = 4;
constexpr int kJacCtaThreads = 128;
constexpr int kJacPairsPerCta = 2;
constexpr int kJacStageRows = 64;                     // rows of the columns staged per Gram chunk
constexpr int kJacPad = kJacCols + 4;

__device__ __forceinline__ void jacobi_cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

struct JacobiPairInfo {
  int bi, bj;
  bool live;
};

__device__ __forceinline__ JacobiPairInfo jacobi_pair_of(const JacobiMat& m, int round, int table) {
  JacobiPairInfo pi{0, 0, false};
  if (table >= m.nblk / 2) return pi;
  round_robin_pair(m.nblk, round, table, pi.bi, pi.bj);
  // (a block beyond L is padding: its columns load as zeros and never rotate; the columns of its partner are
  // still rotated against each other, which is all there is to do when the matrix has a single block)
  pi.live = !(pi.bi * kJacBlock >= m.L && pi.bj * kJacBlock >= m.L);
  return pi;
}

// Shared memory of a CTA, two regions that change hands between the phases of a pair's visit:
//   region 1: Gram: the staged rows (32 x 64 floats, quads swizzled by row so that the 4 x 4 tiles read them
//             without bank conflicts) and two partial Gram matrices; eigensolve: the intermediate Bs = A R;
//             polish: J^T in double precision; apply: the rotations in single precision
//   region 2: eigensolve: As (the Gram matrix, rotated in place) and Js (the accumulated rotation, Js[b][a] =
//             coefficient of old column b in new column a); polish: J^T J - I in the place of As; then the polished
//             rotations in double precision (rows padded to 34)
// The 32 x 32 single-precision matrices have rows of 36 floats: 16-byte rows whose quarter-warp accesses fall into
// different banks.
constexpr int kJacLdD = kJacCols + 2;     // row length of the 32 x 32 double-precision matrices (16-byte rows)
constexpr int kJacLdF = kJacCols + 4;     // the same for the single-precision copy
constexpr size_t kJacStageBytes = sizeof(float) * kJacCols * kJacStageRows;
constexpr size_t kJacMat32Bytes = sizeof(float) * kJacCols * kJacPad;
constexpr size_t kJacMat64Bytes = sizeof(double) * kJacCols * kJacLdD;
constexpr size_t kJacRegion1Bytes = kJacStageBytes + 2 * kJacMat32Bytes;
constexpr size_t kJacRegion2Bytes = 2 * kJacPairsPerCta * kJacMat32Bytes;
static_assert(kJacPairsPerCta * kJacMat64Bytes <= kJacRegion1Bytes, "double-precision J^T fits region 1");
static_assert(kJacPairsPerCta * kJacMat64Bytes <= kJacRegion2Bytes, "double-precision rotations fit region 2");
static_assert(kJacPairsPerCta * kJacMat32Bytes <= kJacRegion1Bytes, "Bs fits region 1");
static_assert(kJacPairsPerCta * sizeof(float) * kJacCols * kJacLdF <= kJacRegion1Bytes, "single-precision rotations fit");

struct JacobiShared {
  __align__(16) unsigned char r1[kJacRegion1Bytes];
  __align__(16) unsigned char r2[kJacRegion2Bytes];
  __align__(16) float2 cs[kJacPairsPerCta][kJacBlock];   // cosine and sine of the 16 rotations of a step
  int active[kJacPairsPerCta];
};

__global__ void __cluster_dims__(kJacCluster, 1, 1) __launch_bounds__(kJacCtaThreads, 5)
jacobi_cluster_kernel(const JacobiMat* mats) {
  extern __shared__ __align__(16) unsigned char jac_smem_raw[];
  JacobiShared& sh = *reinterpret_cast<JacobiShared*>(jac_smem_raw);
  typedef float Mat32[kJacCols][kJacPad];
  typedef double Mat64[kJacCols][kJacLdD];
  typedef float MatF[kJacCols][kJacLdF];
  float* stage = reinterpret_cast<float*>(sh.r1);                               // [32][64], swizzled
  Mat32* Ap = reinterpret_cast<Mat32*>(sh.r1 + kJacStageBytes);                  // [2] partial Gram matrices
  Mat32* Bs = reinterpret_cast<Mat32*>(sh.r1);                                   // [pair]
  Mat64* JTd = reinterpret_cast<Mat64*>(sh.r1);                                  // [pair]
  MatF* Jf = reinterpret_cast<MatF*>(sh.r1);                                     // [pair]
  Mat32* As = reinterpret_cast<Mat32*>(sh.r2);                                   // [pair]; later J^T J - I
  Mat32* Js = reinterpret_cast<Mat32*>(sh.r2 + kJacPairsPerCta * kJacMat32Bytes);  // [pair]
  Mat64* Jd = reinterpret_cast<Mat64*>(sh.r2);                                   // [pair]

  const JacobiMat m = mats[blockIdx.x / kJacCluster];
  const int crank = blockIdx.x % kJacCluster;
  const int tid = threadIdx.x;
  const int L = m.L, ld = m.ld;
  const int tables = m.nblk / 2, rounds = m.nblk - 1;
  const int groups = (tables + kJacCluster * kJacPairsPerCta - 1) / (kJacCluster * kJacPairsPerCta);
  auto global_row = [](const JacobiPairInfo& pi, int a) {
    return (a < kJacBlock ? pi.bi : pi.bj) * kJacBlock + (a & (kJacBlock - 1));
  };

  for (int sweep = 0; sweep < kJacMaxSweeps; ++sweep) {
    for (int round = 0; round < rounds; ++round) {
      for (int grp = 0; grp < groups; ++grp) {
        JacobiPairInfo pis[kJacPairsPerCta];
#pragma unroll
        for (int p = 0; p < kJacPairsPerCta; ++p)
          pis[p] = jacobi_pair_of(m, round, (grp * kJacCluster + crank) * kJacPairsPerCta + p);
        if (!pis[0].live && !pis[1].live) continue;      // the same for every thread of the CTA

        // ---- Gram matrices ----
#pragma unroll 1
        for (int p = 0; p < kJacPairsPerCta; ++p) {
          const JacobiPairInfo pi = pis[p];
          if (!pi.live) {
            if (tid == 0) sh.active[p] = 0;
            continue;
          }
          // 64 tiles of 4 x 4 entries, two groups of threads share the rows of a chunk
          const int kg = tid >> 6, tile = tid & 63, ta = tile >> 3, tb = tile & 7;
          float g[4][4];
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) g[x][y] = 0.f;
          for (int k0 = 0; k0 < ld; k0 += kJacStageRows) {
            __syncthreads();                                // the previous chunk has been consumed
            for (int x = tid; x < kJacCols * (kJacStageRows / 4); x += kJacCtaThreads) {
              const int a = x / (kJacStageRows / 4), q = x % (kJacStageRows / 4);
              const int gr = global_row(pi, a), k = k0 + 4 * q;
              float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
              if (gr < L && k < ld) v = __ldcg(reinterpret_cast<const float4*>(m.XT + static_cast<long long>(gr) * ld + k));
              *reinterpret_cast<float4*>(stage + a * kJacStageRows + 4 * (q ^ ((a >> 2) & 7))) = v;
            }
            __syncthreads();
#pragma unroll 2
            for (int q = kg; q < kJacStageRows / 4; q += 2) {
              float4 a[4], b[4];
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                a[x] = *reinterpret_cast<const float4*>(stage + (4 * ta + x) * kJacStageRows + 4 * (q ^ ta));
                b[x] = *reinterpret_cast<const float4*>(stage + (4 * tb + x) * kJacStageRows + 4 * (q ^ tb));
              }
#pragma unroll
              for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y)
                  g[x][y] += a[x].x * b[y].x + a[x].y * b[y].y + a[x].z * b[y].z + a[x].w * b[y].w;
            }
          }
#pragma unroll
          for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) Ap[kg][4 * ta + x][4 * tb + y] = g[x][y];
          __syncthreads();
          // the two partial matrices added in a fixed order (entry (a, b) and entry (b, a) then agree to the bit); is
          // any pair of columns further from orthogonal than the tolerance?
          auto entry = [&](int a, int b) { return Ap[0][a][b] + Ap[1][a][b]; };
          int any = 0;
          for (int x = tid; x < kJacCols * kJacCols; x += kJacCtaThreads) {
            const int a = x / kJacCols, b = x % kJacCols;
            const float v = a <= b ? entry(a, b) : entry(b, a);
            As[p][a][b] = v;
            if (a < b && v * v > kJacTol * kJacTol * entry(a, a) * entry(b, b)) any = 1;
          }
          any = __syncthreads_or(any);
          if (tid == 0) {
            sh.active[p] = any;
            if (any) atomicOr(m.flags + sweep, 1);
          }
        }
        __syncthreads();
        const bool act0 = sh.active[0] != 0, act1 = sh.active[1] != 0;
        if (!act0 && !act1) continue;                       // the same for every thread of the CTA

        // ---- eigenvectors of the Gram matrices: 64 threads per pair, both pairs in step.  Cyclic two-sided
        // Jacobi in the ordering of Brent and Luk: the 16 rotations of a step act on the columns (and rows) at
        // positions (2i, 2i + 1), and every step ends by moving the columns and rows to the positions of their
        // next partners (position 0 stays, the even positions move up by two, the odd ones down by two, the ends
        // turn around).  After the 31 steps of a sweep every pair has met once and everything is back in its
        // place.  A thread holds 16 consecutive entries of one row, i.e. eight whole pairs, so the column
        // rotation and the move happen in registers (one shuffle with the thread that holds the other half of the
        // row) and all shared-memory traffic is 16-byte accesses. ----
        {
          const int p = tid >> 6, lt = tid & 63;
          const int r = lt >> 1, h = lt & 1;                // this thread: row r, positions 16 h .. 16 h + 15
          const bool mine = p == 0 ? act0 : act1;
          float(&A)[kJacCols][kJacPad] = As[p];
          float(&B)[kJacCols][kJacPad] = Bs[p];
          float(&J)[kJacCols][kJacPad] = Js[p];
          // where row (or column) r goes at the end of a step
          const int r_next = r == 0 ? 0 : (r == 1 ? 2 : (r == kJacCols - 2 ? kJacCols - 1 : ((r & 1) ? r - 2 : r + 2)));
#pragma unroll
          for (int y = 0; y < 16; ++y) J[r][16 * h + y] = (r == 16 * h + y) ? 1.f : 0.f;
          __syncthreads();
          auto load16 = [&](const float* src, float (&v)[16]) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float4 x = *reinterpret_cast<const float4*>(src + 4 * q);
              v[4 * q] = x.x; v[4 * q + 1] = x.y; v[4 * q + 2] = x.z; v[4 * q + 3] = x.w;
            }
          };
          auto store16 = [&](float* dst, const float (&v)[16]) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<float4*>(dst + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          };
          // v <- (v R) moved: rotate the eight pairs, then shift the even entries up and the odd ones down by one
          // pair; the entry that leaves this half of the row is traded for the one that enters it
          auto rotate_and_move = [&](float (&v)[16], const float2 (&c)[8]) {
            float t[16];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              t[2 * i] = c[i].x * v[2 * i] - c[i].y * v[2 * i + 1];
              t[2 * i + 1] = c[i].y * v[2 * i] + c[i].x * v[2 * i + 1];
            }
            const float recv = __shfl_xor_sync(0xffffffffu, h ? t[1] : t[14], 1);
            v[0] = h ? recv : t[0];
            v[2] = h ? t[0] : t[1];
#pragma unroll
            for (int i = 2; i < 8; ++i) v[2 * i] = t[2 * i - 2];
#pragma unroll
            for (int i = 0; i < 7; ++i) v[2 * i + 1] = t[2 * i + 3];
            v[15] = h ? t[14] : recv;
          };
          for (int isweep = 0; isweep < kJacInnerSweeps; ++isweep) {
            int rotated = 0;
            for (int step = 0; step < kJacCols - 1; ++step) {
              if (lt < kJacBlock) {
                const int a = 2 * lt, b = 2 * lt + 1;
                const float aaa = A[a][a], abb = A[b][b], aab = A[a][b];
                float c = 1.f, sn = 0.f;
                if (mine && aab * aab > 1e-12f * aaa * abb && aab != 0.f) {
                  const float tau = (abb - aaa) / (2.f * aab);
                  const float t = (tau >= 0.f ? 1.f : -1.f) / (fabsf(tau) + sqrtf(1.f + tau * tau));
                  c = rsqrtf(1.f + t * t);
                  sn = t * c;
                  rotated = 1;
                }
                sh.cs[p][lt] = make_float2(c, sn);
              }
              __syncthreads();
              float2 c8[8];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const float4 x = *reinterpret_cast<const float4*>(&sh.cs[p][8 * h + 2 * q]);
                c8[2 * q] = make_float2(x.x, x.y);
                c8[2 * q + 1] = make_float2(x.z, x.w);
              }
              float v[16];
              load16(&A[r][16 * h], v);
              rotate_and_move(v, c8);
              store16(&B[r][16 * h], v);                                                   // B = (A R) moved
              load16(&J[r][16 * h], v);
              rotate_and_move(v, c8);
              store16(&J[r][16 * h], v);                                                   // J <- (J R) moved
              __syncthreads();
              const float2 cr = sh.cs[p][r >> 1];
              float w[16];
              load16(&B[r][16 * h], v);
              load16(&B[r ^ 1][16 * h], w);
#pragma unroll
              for (int y = 0; y < 16; ++y) v[y] = (r & 1) ? cr.y * w[y] + cr.x * v[y] : cr.x * v[y] - cr.y * w[y];
              store16(&A[r_next][16 * h], v);                                              // A <- (R^T B) moved
              __syncthreads();
            }
            if (!__syncthreads_or(rotated)) break;
          }
          __syncthreads();
        }

        // ---- the rotations made orthogonal to second order, J <- J (I - (J^T J - I) / 2), in double precision.
        // Thread: pair p, row a, half of the other index.  Operands are widened once, not per product. ----
        {
          const int p = tid >> 6, a = (tid & 63) >> 1, h0 = (tid & 1) * 16;
          for (int x = tid; x < kJacPairsPerCta * kJacCols * kJacCols; x += kJacCtaThreads) {
            const int pp = x / (kJacCols * kJacCols), aa = (x / kJacCols) % kJacCols, bb = x % kJacCols;
            JTd[pp][aa][bb] = static_cast<double>(Js[pp][bb][aa]);
          }
          __syncthreads();
          {
            double row[kJacCols];                                                        // JT[a][.] = column a of J
#pragma unroll
            for (int k = 0; k < kJacCols; k += 2) {
              const double2 v = *reinterpret_cast<const double2*>(&JTd[p][a][k]);
              row[k] = v.x; row[k + 1] = v.y;
            }
#pragma unroll 2
            for (int y = 0; y < 16; ++y) {
              const int b = h0 + y;
              double e = (a == b) ? -1.0 : 0.0;
#pragma unroll
              for (int k = 0; k < kJacCols; k += 2) {
                const double2 v = *reinterpret_cast<const double2*>(&JTd[p][b][k]);
                e += row[k] * v.x + row[k + 1] * v.y;
              }
              As[p][a][b] = static_cast<float>(e);                                       // (J^T J - I)_ab
            }
          }
          __syncthreads();
          {
            double ecol[kJacCols];                                                       // (J^T J - I)[.][a]
#pragma unroll
            for (int k = 0; k < kJacCols; ++k) ecol[k] = static_cast<double>(As[p][k][a]);
            __syncthreads();                                                             // region 2 changes hands
#pragma unroll 2
            for (int y = 0; y < 16; y += 2) {
              const int r = h0 + y;
              double2 acc = *reinterpret_cast<const double2*>(&JTd[p][a][r]);           // J[r][a], J[r + 1][a]
#pragma unroll
              for (int k = 0; k < kJacCols; ++k) {
                const double2 v = *reinterpret_cast<const double2*>(&JTd[p][k][r]);
                acc.x -= 0.5 * v.x * ecol[k];
                acc.y -= 0.5 * v.y * ecol[k];
              }
              *reinterpret_cast<double2*>(&Jd[p][a][r]) = acc;
            }
          }
          __syncthreads();
          for (int x = tid; x < kJacPairsPerCta * kJacCols * kJacCols; x += kJacCtaThreads) {
            const int pp = x / (kJacCols * kJacCols), aa = (x / kJacCols) % kJacCols, bb = x % kJacCols;
            Jf[pp][aa][bb] = static_cast<float>(Jd[pp][aa][bb]);
          }
          __syncthreads();
        }

        // ---- new column a = sum_b J[a][b] (old column b), X in single and V in double precision ----
#pragma unroll 1
        for (int p = 0; p < kJacPairsPerCta; ++p) {
          if (sh.active[p] == 0) continue;
          const JacobiPairInfo pi = pis[p];
          for (int k = tid; k < ld; k += kJacCtaThreads) {
            {
              float x[kJacCols];
#pragma unroll
              for (int b = 0; b < kJacCols; ++b) {
                const int gr = global_row(pi, b);
                x[b] = gr < L ? __ldcg(m.XT + static_cast<long long>(gr) * ld + k) : 0.f;
              }
#pragma unroll 4
              for (int a = 0; a < kJacCols; ++a) {
                float acc = 0.f;
#pragma unroll
                for (int b = 0; b < kJacCols; b += 4) {
                  const float4 j = *reinterpret_cast<const float4*>(&Jf[p][a][b]);
                  acc += j.x * x[b] + j.y * x[b + 1] + j.z * x[b + 2] + j.w * x[b + 3];
                }
                const int gr = global_row(pi, a);
                if (gr < L) m.XT[static_cast<long long>(gr) * ld + k] = acc;
              }
            }
            {
              double v[kJacCols];
#pragma unroll
              for (int b = 0; b < kJacCols; ++b) {
                const int gr = global_row(pi, b);
                v[b] = gr < L ? __ldcg(m.VT + static_cast<long long>(gr) * ld + k) : 0.0;
              }
#pragma unroll 4
              for (int a = 0; a < kJacCols; ++a) {
                double acc = 0.0;
#pragma unroll
                for (int b = 0; b < kJacCols; b += 2) {
                  const double2 j = *reinterpret_cast<const double2*>(&Jd[p][a][b]);
                  acc += j.x * v[b] + j.y * v[b + 1];
                }
                const int gr = global_row(pi, a);
                if (gr < L) m.VT[static_cast<long long>(gr) * ld + k] = acc;
              }
            }
          }
        }
        __syncthreads();     // shared memory is reused by the next group of pairs
      }
      jacobi_cluster_barrier();
    }
    // every rotation of this sweep was flagged before the barrier that ended its last round
    if (__ldcg(m.flags + sweep) == 0) break;
  }
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
    if (lane == 0) {
      nrm[i] = (s == s) ? s : -1.f;   // a norm that is no number goes last: the order below stays total
      rank_of[i] = i;                 // (every entry holds a valid column whatever happens below)
    }
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

// Diagonalise n matrices (descriptors d_mats, already initialised by jacobi_init_kernel).
inline cudaError_t jacobi_batched_launch(const JacobiMat* d_mats, int n, cudaStream_t stream, int64_t* launches) {
  static bool attr_set = false;
  if (!attr_set) {
    const cudaError_t e = cudaFuncSetAttribute(jacobi_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               static_cast<int>(sizeof(JacobiShared)));
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  jacobi_cluster_kernel<<<n * kJacCluster, kJacCtaThreads, sizeof(JacobiShared), stream>>>(d_mats);
  *launches += 1;
  return cudaGetLastError();
}

inline int jacobi_blocks(int L) {
  int nb = (L + kJacBlock - 1) / kJacBlock;
  if (nb < 2) nb = 2;
  return (nb + 1) & ~1;
}

}  // namespace ngalore
