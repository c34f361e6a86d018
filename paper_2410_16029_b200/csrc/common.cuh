// Shared device-side structures of the Natural GaLore step library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ngalore {

constexpr int kMaxHistory = 32;       // s <= 32: one warp lane per Gram row in the solve
constexpr int kStreamThreads = 256;   // threads per CTA of the streaming kernels

// Per-matrix device descriptor (array in device memory, one entry per weight matrix).
struct MatDesc {
  int M, N, rp, s;            // rows, cols, r' = min(r, M, N), history length
  int right;                  // 0: left projection R = P^T G (r' x N); 1: right projection R = G Q (M x r')
  int pr;                     // rows of the projector: M (left) or N (right)
  int lr_rows, lr_cols;       // layout of one low-rank matrix: r' x N (left) or M x ldp (right; columns >= r' stay zero)
  long long rn;               // lr_rows * lr_cols, elements of one low-rank matrix
  int ldp, ldpt;              // leading dimensions of P16 (>= rp) and Pt16 (>= pr), multiples of 8 for TMA
  float* H;                   // history ring: s slots of one low-rank matrix, fp32 (one slot when s == 0); with a
                              // bf16 history only the gradient of the current step (one slot, fp32)
  uint16_t* H16;              // bf16 history ring, s slots (null unless the state keeps its history in bf16)
  float* m;                   // first moment, rp x N (null when the moments are kept in bf16)
  float* v;                   // second moment, rp x N
  uint16_t* m16;              // bf16 moments (null unless the state keeps them in bf16): m rounded to nearest,
  uint16_t* v16;              // v rounded stochastically
  int index;                  // position of the matrix in the state's list (keys the stochastic rounding)
  __half* u16;                // direction u = m / sqrt(v + eps) rounded to fp16, lr_rows x lr_cols
  // Working copies of the projector, both holding the bf16-rounded values of P32 (padding is zero).  The
  // projection GEMM reads bf16 (its other operand G is bf16), the back-projection fp16 (its other operand u is):
  //   left:  P16 (pr x ldp) as fp16 = A of the back-projection;  Pt16 (rp x ldpt) as bf16 = A of the projection
  //   right: P16 (pr x ldp) as bf16 = B of the projection;       Pt16 (rp x ldpt) as fp16 = B of the back-projection
  uint16_t* P16;
  uint16_t* Pt16;
  float* P32;                 // fp32 master of the projector, pr x rp row-major
  double* Kraw;               // s x s raw inner products <H_i, H_j>
  float* wsol;                // kMaxHistory solution weights of (lambda I + K) w = e_cur
  double* gpart;              // per-tile partial Gram rows: ntiles x s
  int* status;                // sticky ngalore_status word
  int* step_bad;              // 1 when this step must leave W, m, v untouched
  int* gram_done;             // fused kernel: count of finished Gram tiles of this step
  int* w_ready;               // fused kernel: set to the step epoch once wsol is valid
  int tile0, ntiles;          // range of streaming tiles owned by this matrix
  int te;                     // elements of one streaming tile of this matrix (multiple of 1024)
};

struct Ctrl {
  long long n_appended;       // low-rank gradients pushed into the ring so far
  long long k;                // optimizer step index
  int epoch;                  // increments every step; flags of the fused kernel compare against it
  int timeout_flag;           // set when a bounded wait ran out
  unsigned int work_counter;  // dynamic tile counter of the fused streaming kernel
  unsigned int gemm_counter0; // dynamic tile counter of the projection GEMM
  unsigned int gemm_counter1; // dynamic tile counter of the back-projection GEMM
  // Testing aids, both cleared at the end of every step.  They exist so that a test can make a bounded wait run
  // out without hanging or trapping anything: the solution of one matrix is computed but not published, and the
  // tiles that wait for it give up after a few polls.
  int spin_limit;             // > 0: polls before a flag wait of the stream kernel is abandoned (0: the default)
  int debug_withhold;         // > 0: the weights of matrix (debug_withhold - 1) are not published in this step
};

struct Hyper {
  float lr, wd, beta1, beta2, eps;
  float pad;
  double lambda;
  unsigned int seed_lo, seed_hi;  // key of the generator behind the stochastic rounding of bf16 second moments
};

// Philox-4x32 with ten rounds (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", 2011).
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, unsigned int k0, unsigned int k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const unsigned int hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const unsigned int hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

// A non-negative float rounded to bf16 up or down with odds in proportion to the distances: sixteen random bits are
// added below the sixteen bits bf16 keeps, and the sum is truncated.
__device__ __forceinline__ unsigned int stochastic_bf16_bits(float x, unsigned int bits16) {
  return (__float_as_uint(x) + bits16) >> 16;
}

struct StreamTile {
  int mat;    // matrix index
  int local;  // tile index inside the matrix
};

// Four floats to four fp16 values (round to nearest even, clamped to the largest finite fp16).
__device__ __forceinline__ uint2 pack_f16x4(float a, float b, float c, float d) {
  constexpr float kMax = 65504.f;
  const __half2 lo = __floats2half2_rn(fminf(fmaxf(a, -kMax), kMax), fminf(fmaxf(b, -kMax), kMax));
  const __half2 hi = __floats2half2_rn(fminf(fmaxf(c, -kMax), kMax), fminf(fmaxf(d, -kMax), kMax));
  uint2 r;
  r.x = *reinterpret_cast<const uint32_t*>(&lo);
  r.y = *reinterpret_cast<const uint32_t*>(&hi);
  return r;
}

// Where the projection writes the low-rank gradient of the current step.
__device__ __forceinline__ float* current_gradient(const MatDesc& d, int cur) {
  return d.H16 != nullptr ? d.H : d.H + static_cast<long long>(cur) * d.rn;
}

__device__ __forceinline__ int ring_cur(const Ctrl* c, int s) {
  return s > 0 ? static_cast<int>(c->n_appended % s) : 0;
}
__device__ __forceinline__ int ring_count(const Ctrl* c, int s) {
  if (s <= 0) return 1;
  long long n = c->n_appended + 1;
  return n < s ? static_cast<int>(n) : s;
}

}  // namespace ngalore
