// C-ABI entry points of the Natural GaLore step library: state layout, orchestration of one
// optimizer step and of the subspace refresh.  See include/ngalore.h for the contract.
#include "../../include/ngalore.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "kernels_refresh.cuh"
#include "kernels_simt_gemm.cuh"
#include "kernels_stream.cuh"
#include "gemm_tcgen05.cuh"
#include "project_tcgen05.cuh"
#include "backproject_tcgen05.cuh"
#include "kernels_fused_stream.cuh"
#include "refresh_tc.cuh"
#include "static_natural_gradient.cuh"
#include "small_rank.cuh"

using namespace ngalore;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct HostMat {
  int M, N, rp;
  bool right;        // projected on the right (short-side rule, M >= N)
  int eM, eN;        // the matrix the refresh sees: G itself (M x N), or G^T with its rows padded to a multiple
                     // of 8 columns (N x eN, eN >= M) when the matrix is projected on the right
  int lr_rows, lr_cols;
  long long rn;
  // refresh scratch (device)
  float *Ya, *Yb, *Xa, *Xb;
  double* C;
  uint16_t* Gt;      // right-projected matrices: G^T as bf16, N x eN (padding columns stay zero)
};

struct BlobHeader {
  uint64_t magic;
  uint64_t arena_bytes;
  int64_t k;
  int64_t n_appended;
  int32_t n, r, s, has_subspace;
  uint64_t shape_hash;
};
constexpr uint64_t kBlobMagic = 0x4E47414C4F524531ull;  // "NGALORE1"

}  // namespace

struct ngalore_state {
  int device = 0;
  int n = 0, r = 0, s = 0, T = 0;
  Hyper hyper{};
  bool hyper_dirty = true;
  ngalore_options opt{};
  std::vector<HostMat> mats;
  std::vector<MatDesc> h_desc;
  MatDesc* d_desc = nullptr;
  char* arena = nullptr;  // persistent optimizer state (exported by checkpoints)
  size_t arena_bytes = 0;
  char* work = nullptr;   // scratch, tables, per-step buffers
  size_t work_bytes = 0;
  Ctrl* d_ctrl = nullptr;
  Hyper* d_hyper = nullptr;
  int* d_status = nullptr;
  int* d_step_bad = nullptr;
  int* d_flags = nullptr;            // gram_done / w_ready of every matrix (scratch, not part of a checkpoint)
  StreamTile* d_tiles = nullptr;
  int n_tiles = 0;
  std::vector<const uint16_t*> refresh_G;  // the gradients as the refresh reads them (G, or its transposed copy)
  // The tensor-core refresh stores rows of r' floats with 16-byte accesses, so it takes the matrices whose r' is a
  // multiple of 4; the rest (r' clipped by a tiny dimension) go through the plain fp64 path.
  std::vector<int> refresh_tc_idx, refresh_plain_idx;
  std::vector<const uint16_t*> refresh_tc_G;
  CholProblem* d_chol = nullptr;
  // Rayleigh-Ritz rotation of the plain refresh path: X of the Jacobi kernels lives in Xa, V (fp64) in C
  JacobiMat* d_jac = nullptr;
  JacobiInit* d_jac_init = nullptr;
  JacobiOut* d_jac_out = nullptr;
  int64_t k = 0;
  int64_t n_appended = 0;
  bool has_subspace = false;         // every matrix has a projector
  std::vector<char> subspace_set;    // per matrix: refreshed or set at least once
  int64_t launches = 0;
  uint64_t shape_hash = 0;
  // tensor-core GEMM plan (tile tables, tensor maps)
  TcPlan tc;
  // fused streaming kernel plan
  FusedPlan fused;
  // tensor-core refresh plan
  RefreshPlan refresh;
  // check and repair of a refreshed basis (finish_refresh): one job per matrix, and the jobs of refresh_tc_idx again
  // in that order
  BasisJob* d_bjobs = nullptr;
  BasisJob* d_bjobs_tc = nullptr;
  double* d_bacc = nullptr;
  // working copies of the projectors of refresh_tc_idx in one launch (finish_refresh)
  WorkingJob* d_wjobs = nullptr;
  int* d_wtile_start = nullptr;
  int n_wjobs = 0, n_wtiles = 0;
  // small-rank path (every r' <= 8): the step as two bandwidth kernels
  SrPlan sr;
  // host-buffer staging; W travels in groups of matrices so that the copies in, the back-projection and the
  // copies out of different groups overlap
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t ev_begin = nullptr, ev_G = nullptr, ev_out = nullptr;
  std::vector<int> group_first;             // first matrix of every group, plus n
  std::vector<cudaEvent_t> ev_w_in, ev_w_done;
  char* stage = nullptr;
  size_t stage_bytes = 0;
  std::vector<float*> stage_W;
  std::vector<uint16_t*> stage_G;
  // update groups: the back-projection runs group by group and records an event after each, so that a consumer of
  // the updated weights (an exchange between ranks, the next forward pass) can start on a group while the next
  // one is still being updated
  std::vector<int> upd_first;               // first matrix of every group, plus n (empty: one launch, no events)
  std::vector<cudaEvent_t> ev_upd;
  // profiling
  bool profiling = false;
  cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
  bool ev_valid = false;
};

namespace {

#define NG_CUDA(expr)                                   \
  do {                                                  \
    cudaError_t e__ = (expr);                           \
    if (e__ != cudaSuccess) return NGALORE_ERR_CUDA;    \
  } while (0)

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

template <int SMAX>
void launch_plain_stream(ngalore_state* st, cudaStream_t stream) {
  if (st->s > 0) {
    gram_kernel<SMAX><<<st->n_tiles, kStreamThreads, 0, stream>>>(st->d_desc, st->d_tiles, st->d_ctrl);
    solve_kernel<<<(st->n + 3) / 4, 128, 0, stream>>>(st->d_desc, st->n, st->d_ctrl, st->d_hyper);
    st->launches += 2;
  }
  combine_kernel<SMAX><<<st->n_tiles, kStreamThreads, 0, stream>>>(st->d_desc, st->d_tiles, st->d_ctrl, st->d_hyper);
  st->launches += 1;
}

ngalore_status upload_hyper(ngalore_state* st, cudaStream_t stream) {
  if (!st->hyper_dirty) return NGALORE_OK;
  NG_CUDA(cudaMemcpyAsync(st->d_hyper, &st->hyper, sizeof(Hyper), cudaMemcpyHostToDevice, stream));
  st->hyper_dirty = false;
  return NGALORE_OK;
}

ngalore_status make_working_copies(ngalore_state* st, int i, cudaStream_t stream) {
  const HostMat& hm = st->mats[i];
  const MatDesc& d = st->h_desc[i];
  dim3 grid((hm.rp + 31) / 32, (hm.eM + 31) / 32), block(32, 8);
  working_copies_kernel<<<grid, block, 0, stream>>>(d.P32, d.P16, d.Pt16, hm.eM, hm.rp, d.ldp, d.ldpt, hm.right ? 0 : 1);
  st->launches += 1;
  NG_CUDA(cudaGetLastError());
  return NGALORE_OK;
}

// Q = orth(Y) for a list of matrices: Gram (fp64) -> batched Cholesky -> Q = Y Lf^-T.
// side 0: Y is M x rp (Ya -> Yb or Yb -> Ya); side 1: Y is N x rp (Xa -> Xb).
ngalore_status orthonormalise(ngalore_state* st, const std::vector<int>& idx, int side, bool from_a,
                              cudaStream_t stream) {
  for (int i : idx) {
    const HostMat& hm = st->mats[i];
    const float* Y = side == 0 ? (from_a ? hm.Ya : hm.Yb) : (from_a ? hm.Xa : hm.Xb);
    const int rows = side == 0 ? hm.eM : hm.eN;
    SimtGemm g{};
    g.m = hm.rp; g.n = hm.rp; g.k = rows;
    g.A = Y; g.a_rs = 1; g.a_cs = hm.rp; g.a_dt = DT_F32;
    g.B = Y; g.b_rs = hm.rp; g.b_cs = 1; g.b_dt = DT_F32;
    g.C = hm.C; g.c_rs = hm.rp; g.c_cs = 1; g.c_dt = DT_F64;
    g.epilogue = EPI_STORE;
    NG_CUDA(launch_simt_gemm<double>(g, stream));
    st->launches += 1;
  }
  // The problem table holds every matrix; launch over the selected ones.
  if (idx.size() == static_cast<size_t>(st->n)) {
    int lmax = 0;
    for (const HostMat& hm : st->mats) lmax = hm.rp > lmax ? hm.rp : lmax;
    NG_CUDA(chol_batched_launch(st->d_chol, st->n, lmax, stream, &st->launches));
  } else {
    for (int i : idx) NG_CUDA(chol_batched_launch(st->d_chol + i, 1, st->mats[i].rp, stream, &st->launches));
  }
  NG_CUDA(cudaGetLastError());
  for (int i : idx) {
    const HostMat& hm = st->mats[i];
    OrthApply p{};
    p.Y = side == 0 ? (from_a ? hm.Ya : hm.Yb) : (from_a ? hm.Xa : hm.Xb);
    p.Q = side == 0 ? (from_a ? hm.Yb : hm.Ya) : (from_a ? hm.Xb : hm.Xa);
    p.Lf = hm.C;
    p.rows = side == 0 ? hm.eM : hm.eN;
    p.L = hm.rp;
    orth_apply_kernel<<<(p.rows + 31) / 32, 256, orth_apply_smem_bytes(p.L), stream>>>(p);
    st->launches += 1;
  }
  NG_CUDA(cudaGetLastError());
  return NGALORE_OK;
}

enum RefreshBuf { BUF_YA, BUF_YB, BUF_XA, BUF_XB };
inline float* refresh_buf(const HostMat& hm, RefreshBuf b) {
  switch (b) {
    case BUF_YA: return hm.Ya;
    case BUF_YB: return hm.Yb;
    case BUF_XA: return hm.Xa;
    default: return hm.Xb;
  }
}

// Y = G X (side 0: out M x rp from X N x rp) or X = G^T Y (side 1: out N x rp from Y M x rp).
ngalore_status apply_gradient(ngalore_state* st, const std::vector<int>& idx, const uint16_t* const* G, int side,
                              RefreshBuf src, RefreshBuf dst, cudaStream_t stream) {
  for (int i : idx) {
    const HostMat& hm = st->mats[i];
    SimtGemm g{};
    if (side == 0) {
      g.m = hm.eM; g.n = hm.rp; g.k = hm.eN;
      g.A = G[i]; g.a_rs = hm.eN; g.a_cs = 1;
    } else {
      g.m = hm.eN; g.n = hm.rp; g.k = hm.eM;
      g.A = G[i]; g.a_rs = 1; g.a_cs = hm.eN;
    }
    g.a_dt = DT_BF16;
    g.B = refresh_buf(hm, src); g.b_rs = hm.rp; g.b_cs = 1; g.b_dt = DT_F32;
    g.C = refresh_buf(hm, dst); g.c_rs = hm.rp; g.c_cs = 1; g.c_dt = DT_F32;
    g.epilogue = EPI_STORE;
    NG_CUDA(launch_simt_gemm<float>(g, stream));
    st->launches += 1;
  }
  return NGALORE_OK;
}

// whole_set: this call completes a refresh of every matrix (even when idx lists only part of them).
// tc_set: idx is the whole list of matrices refreshed on the tensor-core path (ngalore_state::refresh_tc_idx), for
// which the copies of all projectors are one prepared launch.
ngalore_status finish_refresh(ngalore_state* st, const std::vector<int>& idx, bool basis_in_a, cudaStream_t stream,
                              bool whole_set, bool tc_set = false) {
  ngalore_status rc;
  // a basis of zeros (zero gradient) or with entries that are not finite becomes the first r' unit vectors
  NG_CUDA(cudaMemsetAsync(st->d_bacc, 0, sizeof(double) * 2 * st->n, stream));
  if (tc_set) {
    const dim3 grid(32, static_cast<unsigned>(idx.size()));
    basis_check_kernel<<<grid, 256, 0, stream>>>(st->d_bjobs_tc, basis_in_a ? 1 : 0);
    basis_repair_kernel<<<grid, 256, 0, stream>>>(st->d_bjobs_tc, basis_in_a ? 1 : 0);
    st->launches += 2;
  } else {
    for (int i : idx) {
      basis_check_kernel<<<dim3(32, 1), 256, 0, stream>>>(st->d_bjobs + i, basis_in_a ? 1 : 0);
      basis_repair_kernel<<<dim3(32, 1), 256, 0, stream>>>(st->d_bjobs + i, basis_in_a ? 1 : 0);
      st->launches += 2;
    }
  }
  NG_CUDA(cudaGetLastError());
  if (tc_set && basis_in_a && st->n_wjobs > 0) {
    // the whole tensor-core set: master and working copies of every projector in one launch
    working_copies_grouped_kernel<<<st->n_wtiles, dim3(32, 8), 0, stream>>>(st->d_wjobs, st->d_wtile_start, st->n_wjobs);
    st->launches += 1;
    NG_CUDA(cudaGetLastError());
  } else {
    for (int i : idx) {
      const HostMat& hm = st->mats[i];
      NG_CUDA(cudaMemcpyAsync(st->h_desc[i].P32, basis_in_a ? hm.Ya : hm.Yb, sizeof(float) * hm.eM * hm.rp,
                              cudaMemcpyDeviceToDevice, stream));
      if ((rc = make_working_copies(st, i, stream))) return rc;
    }
  }
  if (st->opt.reset_history_on_refresh && whole_set) {
    st->n_appended = 0;
    NG_CUDA(cudaMemsetAsync(&st->d_ctrl->n_appended, 0, sizeof(long long), stream));
  }
  for (int i : idx) st->subspace_set[i] = 1;
  st->has_subspace = true;
  for (char c : st->subspace_set) st->has_subspace = st->has_subspace && c != 0;
  return NGALORE_OK;
}

// Leading columns of the basis that the Rayleigh-Ritz rotation turns into Ritz vectors (see ritz_jacobi.cuh).
inline int ritz_columns(const ngalore_state* st) {
  return st->opt.ritz_columns == 0 ? 256 : (st->opt.ritz_columns < 0 ? (1 << 20) : st->opt.ritz_columns);
}

// Plain SIMT refresh (debug path, and single-matrix refreshes).
ngalore_status refresh_simt(ngalore_state* st, const uint16_t* const* G, const std::vector<int>& idx, int q,
                            cudaStream_t stream) {
  // Random test matrix Omega (N x rp), one hashed stream per matrix and refresh.
  for (int i : idx) {
    const HostMat& hm = st->mats[i];
    const long long cnt = static_cast<long long>(hm.eN) * hm.rp;
    fill_normal_kernel<<<static_cast<unsigned>((cnt + 255) / 256), 256, 0, stream>>>(
        hm.Xa, cnt, st->opt.seed, static_cast<unsigned long long>(st->k) * 65536ull + static_cast<unsigned>(i));
    st->launches += 1;
  }
  NG_CUDA(cudaGetLastError());
  ngalore_status rc;
  // Ya = G Omega; Yb = orth(Ya)
  if ((rc = apply_gradient(st, idx, G, 0, BUF_XA, BUF_YA, stream))) return rc;
  if ((rc = orthonormalise(st, idx, 0, true, stream))) return rc;
  for (int it = 0; it < q; ++it) {
    // Xa = G^T Yb; Xb = orth(Xa); Ya = G Xb; Yb = orth(Ya)
    if ((rc = apply_gradient(st, idx, G, 1, BUF_YB, BUF_XA, stream))) return rc;
    if ((rc = orthonormalise(st, idx, 1, true, stream))) return rc;
    if ((rc = apply_gradient(st, idx, G, 0, BUF_XB, BUF_YA, stream))) return rc;
    if ((rc = orthonormalise(st, idx, 0, true, stream))) return rc;
  }
  // Second pass Yb -> Ya so that a clamped pivot of the first pass cannot leave P non-orthonormal.
  if ((rc = orthonormalise(st, idx, 0, false, stream))) return rc;
  // Rayleigh-Ritz rotation (Sec. 1: P holds the singular vectors): Z = G^T Q into Xa, C = Z^T Z (fp64) into C,
  // eigenvectors V of C by Jacobi rotations (X in Xa; V, fp64, takes over the memory of C once C has been read),
  // V with its columns in falling order of the eigenvalue into Xb (as fp32), Yb = Ya V, and a last
  // orthonormalisation Yb -> Ya (its triangular factor is the identity to about 1e-6, so the columns keep their
  // directions).
  if ((rc = apply_gradient(st, idx, G, 1, BUF_YA, BUF_XA, stream))) return rc;
  for (int i : idx) {
    const HostMat& hm = st->mats[i];
    SimtGemm g{};
    g.m = hm.rp; g.n = hm.rp; g.k = hm.eN;
    g.A = hm.Xa; g.a_rs = 1; g.a_cs = hm.rp; g.a_dt = DT_F32;
    g.B = hm.Xa; g.b_rs = hm.rp; g.b_cs = 1; g.b_dt = DT_F32;
    g.C = hm.C; g.c_rs = hm.rp; g.c_cs = 1; g.c_dt = DT_F64;
    g.epilogue = EPI_STORE;
    NG_CUDA(launch_simt_gemm<double>(g, stream));
    st->launches += 1;
    jacobi_init_kernel<<<1, 256, 0, stream>>>(st->d_jac + i, st->d_jac_init + i);
    st->launches += 1;
    const int Lj = std::min(hm.rp, ritz_columns(st));
    NG_CUDA(jacobi_batched_launch(st->d_jac + i, 1, stream, &st->launches));
    jacobi_finish_kernel<<<dim3(1, kJacFinishSplit), 256, 0, stream>>>(st->d_jac + i, st->d_jac_out + i);
    st->launches += 1;
    SimtGemm a{};
    a.m = hm.eM; a.n = hm.rp; a.k = hm.rp;
    a.A = hm.Ya; a.a_rs = hm.rp; a.a_cs = 1; a.a_dt = DT_F32;
    a.B = hm.Xb; a.b_rs = hm.rp; a.b_cs = 1; a.b_dt = DT_F32;  // the sorted eigenvectors
    a.C = hm.Yb; a.c_rs = hm.rp; a.c_cs = 1; a.c_dt = DT_F32;
    a.epilogue = EPI_STORE;
    NG_CUDA(launch_simt_gemm<float>(a, stream));
    st->launches += 1;
  }
  NG_CUDA(cudaGetLastError());
  if ((rc = orthonormalise(st, idx, 0, false, stream))) return rc;
  return finish_refresh(st, idx, true, stream, idx.size() == static_cast<size_t>(st->n));
}

// The subspace a matrix needs is the leading left one of G (left projection) or the leading right one, i.e. the
// left one of G^T (right projection).  Right-projected matrices get G^T written out once per refresh, so that
// every product below sees a plain row-major matrix of eM x eN.
ngalore_status refresh_impl(ngalore_state* st, const uint16_t* const* G_in, const std::vector<int>& idx,
                            cudaStream_t stream) {
  const int q = st->opt.power_iterations > 0 ? st->opt.power_iterations : 6;
  st->refresh_G.assign(G_in, G_in + st->n);
  for (int i : idx) {
    const HostMat& hm = st->mats[i];
    if (!hm.right) continue;
    dim3 grid((hm.N + 31) / 32, (hm.M + 31) / 32), block(32, 8);
    transpose_bf16_kernel<<<grid, block, 0, stream>>>(G_in[i], hm.Gt, hm.M, hm.N, hm.eN);
    st->launches += 1;
    st->refresh_G[i] = hm.Gt;
  }
  NG_CUDA(cudaGetLastError());
  const uint16_t* const* G = st->refresh_G.data();
  if (st->opt.gemm_impl == 1 || idx.size() != static_cast<size_t>(st->n) || !st->refresh.ready)
    return refresh_simt(st, G, idx, q, stream);
  ngalore_status rc;
  if (!st->refresh_plain_idx.empty() && (rc = refresh_simt(st, G, st->refresh_plain_idx, q, stream))) return rc;
  st->refresh_tc_G.resize(st->refresh_tc_idx.size());
  for (size_t p = 0; p < st->refresh_tc_idx.size(); ++p) st->refresh_tc_G[p] = G[st->refresh_tc_idx[p]];
  if ((rc = refresh_tc_run(st->refresh, st->refresh_tc_G.data(), q, st->opt.seed,
                           static_cast<unsigned long long>(st->k) * 65536ull, st->d_ctrl, stream, &st->launches)))
    return rc;
  // The basis sits in Ya, orthonormal to about 1e-6 where the matrix has enough rows for the bf16-pair rounding
  // of the last product to average out.  Short matrices get one exact pass (Gram, Cholesky and triangular solve in fp64): Ya -> Yb -> Ya.
  std::vector<int> small;
  for (int i : st->refresh_tc_idx)
    if (st->mats[i].eM < 512) small.push_back(i);
  if (!small.empty()) {
    if ((rc = orthonormalise(st, small, 0, true, stream))) return rc;
    for (int i : small) {
      const HostMat& hm = st->mats[i];
      NG_CUDA(cudaMemcpyAsync(hm.Ya, hm.Yb, sizeof(float) * hm.eM * hm.rp, cudaMemcpyDeviceToDevice, stream));
    }
  }
  return finish_refresh(st, st->refresh_tc_idx, true, stream, true, true);
}

// grouped: the caller delivers W in the groups of ngalore_state::group_first; the back-projection of a group waits
// for that group's event ev_w_in and records ev_w_done (host-buffer step, tensor-core path only).
ngalore_status step_impl(ngalore_state* st, float* const* W, const uint16_t* const* G, cudaStream_t stream,
                         bool grouped = false) {
  ngalore_status rc;
  if (st->T > 0 && st->k % st->T == 0) {
    std::vector<int> all(st->n);
    for (int i = 0; i < st->n; ++i) all[i] = i;
    if ((rc = refresh_impl(st, G, all, stream))) return rc;
  }
  if (!st->has_subspace) return NGALORE_ERR_NO_SUBSPACE;
  if ((rc = upload_hyper(st, stream))) return rc;
  if (st->opt.gemm_impl != 1 && (rc = tc_bind_buffers(st->tc, G, W, stream))) return rc;
  const int cur = st->s > 0 ? static_cast<int>(st->n_appended % st->s) : 0;

  if (st->sr.ready && !grouped && st->upd_first.size() <= 1) {
    // small-rank path: projection with the Gram row, then solve + moments + weight update (small_rank.cuh)
    if (st->profiling) NG_CUDA(cudaEventRecord(st->ev[0], stream));
    if ((rc = sr_project_gram(st->sr, st->d_desc, st->tc.d_Gptr, st->d_ctrl, st->s, stream, &st->launches))) return rc;
    if (st->profiling) {
      NG_CUDA(cudaEventRecord(st->ev[1], stream));
      NG_CUDA(cudaEventRecord(st->ev[2], stream));
    }
    if ((rc = sr_update(st->sr, st->d_desc, st->tc.d_Wptr, st->d_ctrl, st->d_hyper, st->s, stream, &st->launches))) return rc;
    advance_kernel<<<1, 1, 0, stream>>>(st->d_ctrl);
    st->launches += 1;
    NG_CUDA(cudaGetLastError());
    if (st->profiling) {
      NG_CUDA(cudaEventRecord(st->ev[3], stream));
      st->ev_valid = true;
    }
    cudaStreamCaptureStatus cap_sr = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap_sr) != cudaSuccess) cap_sr = cudaStreamCaptureStatusNone;
    if (cap_sr == cudaStreamCaptureStatusNone) {
      st->k += 1;
      st->n_appended += 1;
    }
    return NGALORE_OK;
  }
  if (st->profiling) NG_CUDA(cudaEventRecord(st->ev[0], stream));
  // ---- phase 0: R = P^T G into ring slot `cur`
  if (st->opt.gemm_impl == 1) {
    for (int i = 0; i < st->n; ++i) {
      const HostMat& hm = st->mats[i];
      const MatDesc& d = st->h_desc[i];
      SimtGemm g{};
      if (!hm.right) {
        g.m = hm.rp; g.n = hm.N; g.k = hm.M;
        g.A = d.Pt16; g.a_rs = d.ldpt; g.a_cs = 1; g.a_dt = DT_BF16;
        g.B = G[i]; g.b_rs = hm.N; g.b_cs = 1; g.b_dt = DT_BF16;
      } else {
        g.m = hm.M; g.n = hm.rp; g.k = hm.N;
        g.A = G[i]; g.a_rs = hm.N; g.a_cs = 1; g.a_dt = DT_BF16;
        g.B = d.P16; g.b_rs = d.ldp; g.b_cs = 1; g.b_dt = DT_BF16;
      }
      g.C = d.H16 != nullptr ? d.H : d.H + static_cast<long long>(cur) * hm.rn;
      g.c_rs = hm.lr_cols; g.c_cs = 1; g.c_dt = DT_F32;
      g.epilogue = EPI_STORE;
      NG_CUDA(launch_simt_gemm<float>(g, stream));
      st->launches += 1;
    }
  } else {
    if ((rc = tc_project(st->tc, st->d_desc, st->d_ctrl, st->d_hyper, stream, &st->launches))) return rc;
  }
  if (st->profiling) NG_CUDA(cudaEventRecord(st->ev[1], stream));
  // ---- phase 1: Gram row, solve, natural gradient + moments
  if (st->opt.stream_impl == 1) {
    if (st->s <= 8) launch_plain_stream<8>(st, stream);
    else if (st->s <= 16) launch_plain_stream<16>(st, stream);
    else launch_plain_stream<32>(st, stream);
  } else {
    if ((rc = fused_stream_launch(st->fused, st->d_desc, st->n, st->d_ctrl, st->d_hyper, st->s, stream, &st->launches))) return rc;
  }
  NG_CUDA(cudaGetLastError());
  if (st->profiling) NG_CUDA(cudaEventRecord(st->ev[2], stream));
  // ---- phase 2: W <- (1 - lr wd) W - lr P u
  if (st->opt.gemm_impl == 1) {
    for (int i = 0; i < st->n; ++i) {
      const HostMat& hm = st->mats[i];
      const MatDesc& d = st->h_desc[i];
      SimtGemm g{};
      g.m = hm.M; g.n = hm.N; g.k = hm.rp;
      if (!hm.right) {
        g.A = d.P16; g.a_rs = d.ldp; g.a_cs = 1; g.a_dt = DT_F16;
        g.B = d.u16; g.b_rs = hm.N; g.b_cs = 1; g.b_dt = DT_F16;
      } else {
        g.A = d.u16; g.a_rs = hm.lr_cols; g.a_cs = 1; g.a_dt = DT_F16;
        g.B = d.Pt16; g.b_rs = d.ldpt; g.b_cs = 1; g.b_dt = DT_F16;
      }
      g.C = W[i]; g.c_rs = hm.N; g.c_cs = 1; g.c_dt = DT_F32;
      g.epilogue = EPI_W_UPDATE;
      g.hyper = st->d_hyper;
      g.skip_flag = d.step_bad;
      NG_CUDA(launch_simt_gemm<float>(g, stream));
      st->launches += 1;
      for (size_t ug = 0; ug + 1 < st->upd_first.size(); ++ug)
        if (st->upd_first[ug + 1] == i + 1) NG_CUDA(cudaEventRecord(st->ev_upd[ug], stream));
    }
  } else if (grouped) {
    for (size_t g = 0; g + 1 < st->group_first.size(); ++g) {
      NG_CUDA(cudaStreamWaitEvent(stream, st->ev_w_in[g], 0));
      if ((rc = tc_backproject_range(st->tc, st->group_first[g], st->group_first[g + 1], st->d_desc, st->d_ctrl,
                                     st->d_hyper, stream, &st->launches)))
        return rc;
      NG_CUDA(cudaEventRecord(st->ev_w_done[g], stream));
    }
  } else if (st->upd_first.size() > 1) {
    for (size_t ug = 0; ug + 1 < st->upd_first.size(); ++ug) {
      if ((rc = tc_backproject_range(st->tc, st->upd_first[ug], st->upd_first[ug + 1], st->d_desc, st->d_ctrl,
                                     st->d_hyper, stream, &st->launches)))
        return rc;
      NG_CUDA(cudaEventRecord(st->ev_upd[ug], stream));
    }
  } else {
    if ((rc = tc_backproject(st->tc, st->d_desc, st->d_ctrl, st->d_hyper, stream, &st->launches))) return rc;
  }
  advance_kernel<<<1, 1, 0, stream>>>(st->d_ctrl);
  st->launches += 1;
  NG_CUDA(cudaGetLastError());
  if (st->profiling) {
    NG_CUDA(cudaEventRecord(st->ev[3], stream));
    st->ev_valid = true;
  }
  // A call that is being captured into a CUDA graph enqueues nothing yet: the host-side counters then stay where
  // they are (replays advance the device-side counters only; ngalore_poll_status and ngalore_state_export read
  // those back).
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) cap = cudaStreamCaptureStatusNone;
  if (cap == cudaStreamCaptureStatusNone) {
    st->k += 1;
    st->n_appended += 1;
  }
  return NGALORE_OK;
}

}  // namespace

// ======================================================================================= C ABI

extern "C" {

const char* ngalore_status_string(ngalore_status s) {
  switch (s) {
    case NGALORE_OK: return "ok";
    case NGALORE_ERR_INVALID_ARG: return "invalid argument";
    case NGALORE_ERR_ALLOC: return "device allocation failed";
    case NGALORE_ERR_CUDA: return "CUDA runtime error";
    case NGALORE_ERR_UNSUPPORTED_DEVICE: return "unsupported device (compute capability 10.x required)";
    case NGALORE_ERR_NO_SUBSPACE: return "no subspace: refresh or set one first";
    case NGALORE_ERR_NOT_SPD: return "Cholesky pivot not positive";
    case NGALORE_ERR_NONFINITE: return "non-finite value in the Gram matrix";
    case NGALORE_ERR_TIMEOUT: return "a bounded device wait ran out";
  }
  return "unknown status";
}

ngalore_status ngalore_create(const ngalore_shape* shapes, int n_matrices, int r, int s, int T, double lambda,
                              double lr, double beta1, double beta2, double eps, double wd,
                              const ngalore_options* opt, ngalore_state** out) {
  if (out == nullptr) return NGALORE_ERR_INVALID_ARG;
  *out = nullptr;
  if (shapes == nullptr || n_matrices <= 0 || r < 1 || s < 0 || s > kMaxHistory || T < 0) return NGALORE_ERR_INVALID_ARG;
  if (n_matrices > 65535) return NGALORE_ERR_INVALID_ARG;  // grouped launches index the matrix by blockIdx.y
  if (s > 0 && !(lambda > 0.0)) return NGALORE_ERR_INVALID_ARG;
  if (!(beta1 >= 0.0 && beta1 < 1.0 && beta2 >= 0.0 && beta2 < 1.0) || eps < 0.0) return NGALORE_ERR_INVALID_ARG;
  for (int i = 0; i < n_matrices; ++i) {
    if (shapes[i].rows < 1 || shapes[i].cols < 8 || shapes[i].cols % 8 != 0) return NGALORE_ERR_INVALID_ARG;
    if (shapes[i].rows > (1 << 24) || shapes[i].cols > (1 << 24)) return NGALORE_ERR_INVALID_ARG;
  }
  if (opt != nullptr && opt->struct_size != static_cast<int32_t>(sizeof(ngalore_options))) return NGALORE_ERR_INVALID_ARG;
  if (opt != nullptr && (opt->projection_rule < 0 || opt->projection_rule > 1)) return NGALORE_ERR_INVALID_ARG;
  if (opt != nullptr && (opt->history_bf16 < 0 || opt->history_bf16 > 1)) return NGALORE_ERR_INVALID_ARG;
  if (opt != nullptr && (opt->gram_fusion < 0 || opt->gram_fusion > 1)) return NGALORE_ERR_INVALID_ARG;
  if (opt != nullptr && opt->ritz_columns < -1) return NGALORE_ERR_INVALID_ARG;
  if (opt != nullptr && (opt->small_rank_path < 0 || opt->small_rank_path > 1)) return NGALORE_ERR_INVALID_ARG;
  // bf16 moments live in the fused stream kernel only; the rounding stream is keyed by the element's position in
  // the unpadded low-rank matrix, which the padded layout of right-projected matrices does not keep
  if (opt != nullptr && (opt->moments_bf16 < 0 || opt->moments_bf16 > 1)) return NGALORE_ERR_INVALID_ARG;
  if (opt != nullptr && opt->moments_bf16 == 1 && (opt->stream_impl == 1 || opt->projection_rule == 1)) return NGALORE_ERR_INVALID_ARG;
  // the bf16 history lives in the fused stream kernel only
  if (opt != nullptr && opt->history_bf16 == 1 && (s < 1 || opt->stream_impl == 1)) return NGALORE_ERR_INVALID_ARG;

  int dev = 0;
  NG_CUDA(cudaGetDevice(&dev));
  cudaDeviceProp prop{};
  NG_CUDA(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return NGALORE_ERR_UNSUPPORTED_DEVICE;

  ngalore_state* st = new (std::nothrow) ngalore_state();
  if (st == nullptr) return NGALORE_ERR_ALLOC;
  st->device = dev;
  st->n = n_matrices; st->r = r; st->s = s; st->T = T;
  st->hyper.lr = static_cast<float>(lr); st->hyper.wd = static_cast<float>(wd);
  st->hyper.beta1 = static_cast<float>(beta1); st->hyper.beta2 = static_cast<float>(beta2);
  st->hyper.eps = static_cast<float>(eps); st->hyper.lambda = lambda;
  if (opt != nullptr) st->opt = *opt;
  st->opt.struct_size = sizeof(ngalore_options);
  if (st->opt.seed == 0) st->opt.seed = 0x9E3779B97F4A7C15ull;
  st->hyper.seed_lo = static_cast<unsigned int>(st->opt.seed & 0xFFFFFFFFull);
  st->hyper.seed_hi = static_cast<unsigned int>(st->opt.seed >> 32);

  // ---- streaming tile size.  A work item of the persistent stream kernel carries a fixed cost (table and
  // descriptor loads, the end-of-tile reduction, the completion counter), so tiles are large; measured on the
  // 1.1B shapes, 65536 to 262144 elements are within 1 % of each other and 16384 costs 4 %.  Tiles shrink only to
  // keep about two items per pass and SM on small models.  The history is read from HBM twice per step: a big
  // matrix's history does not survive in L2 between the Gram pass and the combination pass.
  uint64_t hash = 1469598103934665603ull;
  st->mats.resize(n_matrices);
  long long total_rn = 0;
  for (int i = 0; i < n_matrices; ++i) {
    HostMat& hm = st->mats[i];
    hm.M = static_cast<int>(shapes[i].rows); hm.N = static_cast<int>(shapes[i].cols);
    hm.rp = r < hm.M ? r : hm.M;
    if (hm.N < hm.rp) hm.rp = hm.N;
    hm.right = st->opt.projection_rule == 1 && hm.M >= hm.N;
    const int ldr = (hm.rp + 7) / 8 * 8;
    hm.eM = hm.right ? hm.N : hm.M;
    hm.eN = hm.right ? (hm.M + 7) / 8 * 8 : hm.N;
    hm.lr_rows = hm.right ? hm.M : hm.rp;
    hm.lr_cols = hm.right ? ldr : hm.N;
    hm.rn = static_cast<long long>(hm.lr_rows) * hm.lr_cols;
    hm.Gt = nullptr;
    total_rn += hm.rn;
    hash = (hash ^ static_cast<uint64_t>(hm.M)) * 1099511628211ull;
    hash = (hash ^ static_cast<uint64_t>(hm.N)) * 1099511628211ull;
    hash = (hash ^ static_cast<uint64_t>((hm.right ? 2 : 1) + (st->opt.history_bf16 ? 4 : 0) + (st->opt.moments_bf16 ? 8 : 0))) * 1099511628211ull;
  }
  st->shape_hash = hash;
  // Stream tiles: two per SM and pass on large workloads.  Where that would make them short, one per SM: every tile
  // ends with a block-wide reduction and a handful of global round trips, which on small workloads weigh as much
  // as its traffic (measured, stream phase: RoBERTa-base shapes r = 8 / r = 4 68 -> 44 us / 52 -> 39 us, 60M shapes
  // 116 -> 106 us; the 130M shapes and larger are 2 % better with two).
  long long te_all = total_rn / (2ll * prop.multiProcessorCount) / 1024 * 1024;
  if (te_all < 32768) te_all *= 2;
  if (te_all < 4096) te_all = 4096;
  if (te_all > 131072) te_all = 131072;
  std::vector<int> tile_elems(n_matrices, static_cast<int>(te_all));
  // The matrices at the end of the item list get tiles a quarter of the size, so that the last wave of the
  // kernel ends more evenly (the tail of one full-size tile per SM is about 0.1 ms on the 1.1B shapes).
  if (te_all >= 32768) {
    const long long tail_budget = static_cast<long long>(prop.multiProcessorCount) * te_all;
    long long acc = 0;
    for (int i = n_matrices - 1; i >= 0 && acc < tail_budget; --i) {
      tile_elems[i] = static_cast<int>(te_all / 4 / 1024 * 1024);
      acc += st->mats[i].rn;
    }
  }

  // ---- arena layout
  const int slots = s > 0 ? s : 1;
  const bool hist16 = st->opt.history_bf16 == 1;
  const bool mom16 = st->opt.moments_bf16 == 1;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  struct Offs { size_t H, m, v, P32, P16, Pt16, Kraw, wsol; };
  std::vector<Offs> offs(n_matrices);
  const size_t o_ctrl = take(sizeof(Ctrl));
  const size_t o_status = take(sizeof(int) * n_matrices);
  const size_t o_bad = take(sizeof(int) * n_matrices);
  for (int i = 0; i < n_matrices; ++i) {
    const HostMat& hm = st->mats[i];
    offs[i].H = hist16 ? take(sizeof(uint16_t) * hm.rn * slots) : take(sizeof(float) * hm.rn * slots);
    offs[i].m = take((mom16 ? sizeof(uint16_t) : sizeof(float)) * hm.rn);
    offs[i].v = take((mom16 ? sizeof(uint16_t) : sizeof(float)) * hm.rn);
    offs[i].P32 = take(sizeof(float) * hm.eM * hm.rp);
    offs[i].P16 = take(sizeof(uint16_t) * hm.eM * ((hm.rp + 7) / 8 * 8));
    offs[i].Pt16 = take(sizeof(uint16_t) * hm.rp * ((hm.eM + 7) / 8 * 8));
    offs[i].Kraw = take(sizeof(double) * slots * slots);
    offs[i].wsol = take(sizeof(float) * kMaxHistory);
  }
  st->arena_bytes = off;

  // ---- work layout
  off = 0;
  struct WOffs { size_t u16, gpart, Ya, Yb, Xa, Xb, C, Gt, Rcur; };
  std::vector<WOffs> woffs(n_matrices);
  const size_t o_hyper = take(sizeof(Hyper));
  const size_t o_desc = take(sizeof(MatDesc) * n_matrices);
  const size_t o_chol = take(sizeof(CholProblem) * n_matrices);
  const size_t o_flags = take(sizeof(int) * 2 * n_matrices);
  const size_t o_jac = take(sizeof(JacobiMat) * n_matrices);
  const size_t o_jac_init = take(sizeof(JacobiInit) * n_matrices);
  const size_t o_jac_out = take(sizeof(JacobiOut) * n_matrices);
  const size_t o_jac_flags = take(sizeof(int) * kJacMaxSweeps * n_matrices);
  int n_tiles = 0;
  std::vector<StreamTile> tiles;
  std::vector<int> tile0(n_matrices), ntl(n_matrices);
  for (int i = 0; i < n_matrices; ++i) {
    const HostMat& hm = st->mats[i];
    const int te = tile_elems[i];
    ntl[i] = static_cast<int>((hm.rn + te - 1) / te);
    tile0[i] = n_tiles;
    for (int t = 0; t < ntl[i]; ++t) tiles.push_back(StreamTile{i, t});
    n_tiles += ntl[i];
    woffs[i].u16 = take(sizeof(__half) * hm.rn);
    woffs[i].gpart = take(sizeof(double) * ntl[i] * slots * (hist16 ? 2 : 1));
    woffs[i].Rcur = hist16 ? take(sizeof(float) * hm.rn) : 0;
    woffs[i].Ya = take(sizeof(float) * hm.eM * hm.rp);
    woffs[i].Yb = take(sizeof(float) * hm.eM * hm.rp);
    woffs[i].Xa = take(sizeof(float) * hm.eN * hm.rp);
    woffs[i].Xb = take(sizeof(float) * hm.eN * hm.rp);
    woffs[i].C = take(sizeof(double) * hm.rp * ((hm.rp + 3) / 4 * 4));
    woffs[i].Gt = hm.right ? take(sizeof(uint16_t) * hm.N * hm.eN) : 0;
  }
  st->n_tiles = n_tiles;
  const size_t o_tiles = take(sizeof(StreamTile) * n_tiles);
  st->work_bytes = off;

  auto fail = [&](ngalore_status code) {
    ngalore_destroy(st);
    return code;
  };
  if (cudaMalloc(&st->arena, st->arena_bytes) != cudaSuccess) { st->arena = nullptr; return fail(NGALORE_ERR_ALLOC); }
  if (cudaMalloc(&st->work, st->work_bytes) != cudaSuccess) { st->work = nullptr; return fail(NGALORE_ERR_ALLOC); }
  if (cudaMemset(st->arena, 0, st->arena_bytes) != cudaSuccess) return fail(NGALORE_ERR_CUDA);
  if (cudaMemset(st->work, 0, st->work_bytes) != cudaSuccess) return fail(NGALORE_ERR_CUDA);

  st->d_ctrl = reinterpret_cast<Ctrl*>(st->arena + o_ctrl);
  st->d_status = reinterpret_cast<int*>(st->arena + o_status);
  st->d_step_bad = reinterpret_cast<int*>(st->arena + o_bad);
  st->d_hyper = reinterpret_cast<Hyper*>(st->work + o_hyper);
  st->d_desc = reinterpret_cast<MatDesc*>(st->work + o_desc);
  st->d_chol = reinterpret_cast<CholProblem*>(st->work + o_chol);
  st->d_tiles = reinterpret_cast<StreamTile*>(st->work + o_tiles);
  int* flags = reinterpret_cast<int*>(st->work + o_flags);
  st->d_flags = flags;
  st->d_jac = reinterpret_cast<JacobiMat*>(st->work + o_jac);
  st->d_jac_init = reinterpret_cast<JacobiInit*>(st->work + o_jac_init);
  st->d_jac_out = reinterpret_cast<JacobiOut*>(st->work + o_jac_out);
  std::vector<JacobiMat> jac(n_matrices);
  std::vector<JacobiInit> jac_init(n_matrices);
  std::vector<JacobiOut> jac_out(n_matrices);
  st->subspace_set.assign(n_matrices, 0);

  st->h_desc.resize(n_matrices);
  std::vector<CholProblem> chol(n_matrices);
  std::vector<float> w_init(kMaxHistory, 0.f);
  w_init[0] = 1.f;
  for (int i = 0; i < n_matrices; ++i) {
    HostMat& hm = st->mats[i];
    MatDesc& d = st->h_desc[i];
    d.M = hm.M; d.N = hm.N; d.rp = hm.rp; d.s = s; d.rn = hm.rn;
    d.right = hm.right ? 1 : 0; d.pr = hm.eM; d.lr_rows = hm.lr_rows; d.lr_cols = hm.lr_cols;
    d.ldp = (hm.rp + 7) / 8 * 8; d.ldpt = (hm.eM + 7) / 8 * 8;
    if (hist16) {
      d.H16 = reinterpret_cast<uint16_t*>(st->arena + offs[i].H);
      d.H = reinterpret_cast<float*>(st->work + woffs[i].Rcur);
    } else {
      d.H16 = nullptr;
      d.H = reinterpret_cast<float*>(st->arena + offs[i].H);
    }
    d.index = i;
    if (mom16) {
      d.m = nullptr; d.v = nullptr;
      d.m16 = reinterpret_cast<uint16_t*>(st->arena + offs[i].m);
      d.v16 = reinterpret_cast<uint16_t*>(st->arena + offs[i].v);
    } else {
      d.m = reinterpret_cast<float*>(st->arena + offs[i].m);
      d.v = reinterpret_cast<float*>(st->arena + offs[i].v);
      d.m16 = nullptr; d.v16 = nullptr;
    }
    d.P32 = reinterpret_cast<float*>(st->arena + offs[i].P32);
    d.P16 = reinterpret_cast<uint16_t*>(st->arena + offs[i].P16);
    d.Pt16 = reinterpret_cast<uint16_t*>(st->arena + offs[i].Pt16);
    d.Kraw = reinterpret_cast<double*>(st->arena + offs[i].Kraw);
    d.wsol = reinterpret_cast<float*>(st->arena + offs[i].wsol);
    d.u16 = reinterpret_cast<__half*>(st->work + woffs[i].u16);
    d.gpart = reinterpret_cast<double*>(st->work + woffs[i].gpart);
    d.status = st->d_status + i;
    d.step_bad = st->d_step_bad + i;
    d.gram_done = flags + 2 * i;
    d.w_ready = flags + 2 * i + 1;
    d.tile0 = tile0[i]; d.ntiles = ntl[i]; d.te = tile_elems[i];
    hm.Ya = reinterpret_cast<float*>(st->work + woffs[i].Ya);
    hm.Yb = reinterpret_cast<float*>(st->work + woffs[i].Yb);
    hm.Xa = reinterpret_cast<float*>(st->work + woffs[i].Xa);
    hm.Xb = reinterpret_cast<float*>(st->work + woffs[i].Xb);
    hm.C = reinterpret_cast<double*>(st->work + woffs[i].C);
    if (hm.right) hm.Gt = reinterpret_cast<uint16_t*>(st->work + woffs[i].Gt);
    chol[i].C = hm.C; chol[i].L = hm.rp; chol[i].pad = 0; chol[i].tiny = 0.0;
    // eN >= r' and a multiple of 8, so r' rows of ld <= eN floats fit in the eN x r' floats of Xa; V (r' x ld
    // doubles) takes over C, which is allocated with that leading dimension
    const int Lj = std::min(hm.rp, ritz_columns(st));
    jac[i] = JacobiMat{hm.Xa, hm.C, Lj, (Lj + 3) & ~3, jacobi_blocks(Lj),
                       reinterpret_cast<int*>(st->work + o_jac_flags) + kJacMaxSweeps * i};
    jac_init[i] = JacobiInit{nullptr, hm.C, hm.rp};
    jac_out[i] = JacobiOut{hm.Xb, hm.rp, nullptr, nullptr, 0, hm.rp};
    if (s == 0 && cudaMemcpy(d.wsol, w_init.data(), sizeof(float) * kMaxHistory, cudaMemcpyHostToDevice) != cudaSuccess)
      return fail(NGALORE_ERR_CUDA);
  }
  if (cudaMemcpy(st->d_desc, st->h_desc.data(), sizeof(MatDesc) * n_matrices, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(st->d_chol, chol.data(), sizeof(CholProblem) * n_matrices, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(st->d_tiles, tiles.data(), sizeof(StreamTile) * n_tiles, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(st->d_hyper, &st->hyper, sizeof(Hyper), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(st->d_jac, jac.data(), sizeof(JacobiMat) * n_matrices, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(st->d_jac_init, jac_init.data(), sizeof(JacobiInit) * n_matrices, cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(st->d_jac_out, jac_out.data(), sizeof(JacobiOut) * n_matrices, cudaMemcpyHostToDevice) != cudaSuccess)
    return fail(NGALORE_ERR_CUDA);
  st->hyper_dirty = false;

  // kernels with large dynamic shared memory
  int max_rp = 0;
  for (const HostMat& hm : st->mats) max_rp = hm.rp > max_rp ? hm.rp : max_rp;
  if (orth_apply_smem_bytes(max_rp) > static_cast<size_t>(prop.sharedMemPerBlockOptin)) return fail(NGALORE_ERR_INVALID_ARG);
  if (cudaFuncSetAttribute(orth_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(orth_apply_smem_bytes(max_rp))) != cudaSuccess)
    return fail(NGALORE_ERR_CUDA);

  const bool allow_gram_fusion = st->opt.gemm_impl != 1 && st->opt.stream_impl != 1 && !hist16 && st->opt.gram_fusion == 1;
  ngalore_status rc = tc_plan_create(st->tc, st->h_desc, st->d_desc, s, prop.multiProcessorCount, allow_gram_fusion);
  if (rc != NGALORE_OK) return fail(rc);
  if ((rc = tc_project_init()) != NGALORE_OK) return fail(rc);
  if ((rc = tc_backproject_init()) != NGALORE_OK) return fail(rc);
  rc = fused_plan_create(st->fused, st->h_desc, s, prop.multiProcessorCount, &st->tc.gram_fused);
  if (rc != NGALORE_OK) return fail(rc);
  if (st->opt.gemm_impl != 1 && st->opt.stream_impl != 1 && st->opt.gram_fusion != 1 && st->opt.small_rank_path == 1 &&
      sr_eligible(st->h_desc, s)) {
    rc = sr_plan_create(st->sr, st->h_desc, s, prop.multiProcessorCount);
    if (rc != NGALORE_OK) return fail(rc);
  }
  if (st->opt.gemm_impl != 1) {
    // the refresh plan sees every matrix it takes in the orientation whose left subspace is wanted
    std::vector<float*> Yf, Zf;
    std::vector<MatDesc> eff;
    for (int i = 0; i < n_matrices; ++i) {
      if (st->mats[i].rp % 4 != 0) { st->refresh_plain_idx.push_back(i); continue; }
      st->refresh_tc_idx.push_back(i);
      Yf.push_back(st->mats[i].Ya); Zf.push_back(st->mats[i].Xa);
      eff.push_back(st->h_desc[i]);
      eff.back().M = st->mats[i].eM; eff.back().N = st->mats[i].eN;
    }
    if (!eff.empty()) {
      rc = refresh_plan_create(st->refresh, eff, Yf, Zf, prop.multiProcessorCount, ritz_columns(st));
      if (rc != NGALORE_OK) return fail(rc);
      std::vector<WorkingJob> jobs;
      std::vector<int> start(1, 0);
      for (int i : st->refresh_tc_idx) {
        const HostMat& hm = st->mats[i];
        const MatDesc& d = st->h_desc[i];
        const int tx = (hm.rp + 31) / 32, ty = (hm.eM + 31) / 32;
        jobs.push_back(WorkingJob{hm.Ya, d.P32, d.P16, d.Pt16, hm.eM, hm.rp, d.ldp, d.ldpt, hm.right ? 0 : 1, tx});
        start.push_back(start.back() + tx * ty);
      }
      st->n_wjobs = static_cast<int>(jobs.size());
      st->n_wtiles = start.back();
      if (cudaMalloc(&st->d_wjobs, sizeof(WorkingJob) * jobs.size()) != cudaSuccess ||
          cudaMalloc(&st->d_wtile_start, sizeof(int) * start.size()) != cudaSuccess)
        return fail(NGALORE_ERR_ALLOC);
      if (cudaMemcpy(st->d_wjobs, jobs.data(), sizeof(WorkingJob) * jobs.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
          cudaMemcpy(st->d_wtile_start, start.data(), sizeof(int) * start.size(), cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(NGALORE_ERR_CUDA);
    }
  }
  {
    if (cudaMalloc(&st->d_bacc, sizeof(double) * 2 * n_matrices) != cudaSuccess ||
        cudaMalloc(&st->d_bjobs, sizeof(BasisJob) * n_matrices) != cudaSuccess ||
        cudaMalloc(&st->d_bjobs_tc, sizeof(BasisJob) * (st->refresh_tc_idx.size() + 1)) != cudaSuccess)
      return fail(NGALORE_ERR_ALLOC);
    std::vector<BasisJob> jobs(n_matrices), jobs_tc;
    for (int i = 0; i < n_matrices; ++i) {
      const HostMat& hm = st->mats[i];
      jobs[i] = BasisJob{hm.Ya, hm.Yb, st->d_bacc + 2 * i, st->d_status + i, hm.eM, hm.rp};
    }
    for (int i : st->refresh_tc_idx) jobs_tc.push_back(jobs[i]);
    if (cudaMemcpy(st->d_bjobs, jobs.data(), sizeof(BasisJob) * jobs.size(), cudaMemcpyHostToDevice) != cudaSuccess ||
        (!jobs_tc.empty() && cudaMemcpy(st->d_bjobs_tc, jobs_tc.data(), sizeof(BasisJob) * jobs_tc.size(),
                                        cudaMemcpyHostToDevice) != cudaSuccess))
      return fail(NGALORE_ERR_CUDA);
  }
  for (int e = 0; e < 4; ++e)
    if (cudaEventCreate(&st->ev[e]) != cudaSuccess) return fail(NGALORE_ERR_CUDA);
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(NGALORE_ERR_CUDA);
  *out = st;
  return NGALORE_OK;
}

void ngalore_destroy(ngalore_state* st) {
  if (st == nullptr) return;
  DeviceGuard guard(st->device);
  cudaDeviceSynchronize();
  tc_plan_destroy(st->tc);
  fused_plan_destroy(st->fused);
  refresh_plan_destroy(st->refresh);
  sr_plan_destroy(st->sr);
  for (int e = 0; e < 4; ++e)
    if (st->ev[e]) cudaEventDestroy(st->ev[e]);
  for (cudaEvent_t e : st->ev_upd) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : st->ev_w_in) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : st->ev_w_done) if (e) cudaEventDestroy(e);
  if (st->ev_begin) cudaEventDestroy(st->ev_begin);
  if (st->ev_G) cudaEventDestroy(st->ev_G);
  if (st->ev_out) cudaEventDestroy(st->ev_out);
  if (st->copy_in) cudaStreamDestroy(st->copy_in);
  if (st->copy_out) cudaStreamDestroy(st->copy_out);
  if (st->stage) cudaFree(st->stage);
  if (st->work) cudaFree(st->work);
  if (st->d_bjobs) cudaFree(st->d_bjobs);
  if (st->d_bjobs_tc) cudaFree(st->d_bjobs_tc);
  if (st->d_bacc) cudaFree(st->d_bacc);
  if (st->d_wjobs) cudaFree(st->d_wjobs);
  if (st->d_wtile_start) cudaFree(st->d_wtile_start);
  if (st->arena) cudaFree(st->arena);
  delete st;
}

ngalore_status ngalore_step(ngalore_state* st, float* const* W, const uint16_t* const* G, void* stream) {
  if (st == nullptr || W == nullptr || G == nullptr) return NGALORE_ERR_INVALID_ARG;
  for (int i = 0; i < st->n; ++i) {
    if (W[i] == nullptr || G[i] == nullptr) return NGALORE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(W[i]) | reinterpret_cast<uintptr_t>(G[i])) & 15u) return NGALORE_ERR_INVALID_ARG;
  }
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  return step_impl(st, W, G, static_cast<cudaStream_t>(stream));
}

ngalore_status ngalore_refresh_subspace(ngalore_state* st, const uint16_t* const* G, int matrix_index, void* stream) {
  if (st == nullptr || G == nullptr || matrix_index < -1 || matrix_index >= st->n) return NGALORE_ERR_INVALID_ARG;
  std::vector<int> idx;
  if (matrix_index < 0) {
    for (int i = 0; i < st->n; ++i) idx.push_back(i);
  } else {
    idx.push_back(matrix_index);
  }
  for (int i : idx)
    if (G[i] == nullptr || (reinterpret_cast<uintptr_t>(G[i]) & 15u)) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  return refresh_impl(st, G, idx, static_cast<cudaStream_t>(stream));
}

ngalore_status ngalore_step_host(ngalore_state* st, float* const* W_host, const uint16_t* const* G_host, void* stream) {
  if (st == nullptr || W_host == nullptr || G_host == nullptr) return NGALORE_ERR_INVALID_ARG;
  for (int i = 0; i < st->n; ++i)
    if (W_host[i] == nullptr || G_host[i] == nullptr) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (st->stage == nullptr) {
    size_t off = 0;
    std::vector<size_t> ow(st->n), og(st->n);
    for (int i = 0; i < st->n; ++i) {
      const size_t mn = static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
      ow[i] = off; off += align_up(mn * sizeof(float));
      og[i] = off; off += align_up(mn * sizeof(uint16_t));
    }
    if (cudaMalloc(&st->stage, off) != cudaSuccess) { st->stage = nullptr; return NGALORE_ERR_ALLOC; }
    st->stage_bytes = off;
    st->stage_W.resize(st->n); st->stage_G.resize(st->n);
    for (int i = 0; i < st->n; ++i) {
      st->stage_W[i] = reinterpret_cast<float*>(st->stage + ow[i]);
      st->stage_G[i] = reinterpret_cast<uint16_t*>(st->stage + og[i]);
    }
  }
  if (st->opt.gemm_impl == 1) {
    // debug path: everything in order on the caller's stream
    for (int i = 0; i < st->n; ++i) {
      const size_t mn = static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
      NG_CUDA(cudaMemcpyAsync(st->stage_G[i], G_host[i], mn * sizeof(uint16_t), cudaMemcpyHostToDevice, s));
      NG_CUDA(cudaMemcpyAsync(st->stage_W[i], W_host[i], mn * sizeof(float), cudaMemcpyHostToDevice, s));
    }
    ngalore_status rc = step_impl(st, st->stage_W.data(), st->stage_G.data(), s);
    if (rc != NGALORE_OK) return rc;
    for (int i = 0; i < st->n; ++i) {
      const size_t mn = static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
      NG_CUDA(cudaMemcpyAsync(W_host[i], st->stage_W[i], mn * sizeof(float), cudaMemcpyDeviceToHost, s));
    }
    NG_CUDA(cudaStreamSynchronize(s));
    return NGALORE_OK;
  }
  // Pipelined: only the back-projection touches W, so the gradients go in first and the projection and the
  // history phase run while W is still arriving; W then moves in about eight groups of matrices, each group's
  // copy in, back-projection and copy out chained by events, so that the two directions of the link overlap.
  if (st->copy_in == nullptr) {
    NG_CUDA(cudaStreamCreateWithFlags(&st->copy_in, cudaStreamNonBlocking));
    NG_CUDA(cudaStreamCreateWithFlags(&st->copy_out, cudaStreamNonBlocking));
    NG_CUDA(cudaEventCreateWithFlags(&st->ev_begin, cudaEventDisableTiming));
    NG_CUDA(cudaEventCreateWithFlags(&st->ev_G, cudaEventDisableTiming));
    NG_CUDA(cudaEventCreateWithFlags(&st->ev_out, cudaEventDisableTiming));
    size_t total = 0;
    for (const HostMat& hm : st->mats) total += static_cast<size_t>(hm.M) * hm.N;
    const int want = st->n < 8 ? st->n : 8;
    st->group_first.assign(1, 0);
    size_t acc = 0;
    for (int i = 0; i < st->n; ++i) {
      acc += static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
      const size_t done_groups = st->group_first.size();
      if (i + 1 < st->n && static_cast<int>(done_groups) < want && acc * want >= total * done_groups)
        st->group_first.push_back(i + 1);
    }
    st->group_first.push_back(st->n);
    const size_t ng = st->group_first.size() - 1;
    st->ev_w_in.resize(ng); st->ev_w_done.resize(ng);
    for (size_t g = 0; g < ng; ++g) {
      NG_CUDA(cudaEventCreateWithFlags(&st->ev_w_in[g], cudaEventDisableTiming));
      NG_CUDA(cudaEventCreateWithFlags(&st->ev_w_done[g], cudaEventDisableTiming));
    }
  }
  const size_t ng = st->group_first.size() - 1;
  NG_CUDA(cudaEventRecord(st->ev_begin, s));
  NG_CUDA(cudaStreamWaitEvent(st->copy_in, st->ev_begin, 0));
  for (int i = 0; i < st->n; ++i) {
    const size_t mn = static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
    NG_CUDA(cudaMemcpyAsync(st->stage_G[i], G_host[i], mn * sizeof(uint16_t), cudaMemcpyHostToDevice, st->copy_in));
  }
  NG_CUDA(cudaEventRecord(st->ev_G, st->copy_in));
  for (size_t g = 0; g < ng; ++g) {
    for (int i = st->group_first[g]; i < st->group_first[g + 1]; ++i) {
      const size_t mn = static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
      NG_CUDA(cudaMemcpyAsync(st->stage_W[i], W_host[i], mn * sizeof(float), cudaMemcpyHostToDevice, st->copy_in));
    }
    NG_CUDA(cudaEventRecord(st->ev_w_in[g], st->copy_in));
  }
  NG_CUDA(cudaStreamWaitEvent(s, st->ev_G, 0));
  ngalore_status rc = step_impl(st, st->stage_W.data(), st->stage_G.data(), s, true);
  if (rc != NGALORE_OK) {
    cudaStreamSynchronize(st->copy_in);
    return rc;
  }
  for (size_t g = 0; g < ng; ++g) {
    NG_CUDA(cudaStreamWaitEvent(st->copy_out, st->ev_w_done[g], 0));
    for (int i = st->group_first[g]; i < st->group_first[g + 1]; ++i) {
      const size_t mn = static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
      NG_CUDA(cudaMemcpyAsync(W_host[i], st->stage_W[i], mn * sizeof(float), cudaMemcpyDeviceToHost, st->copy_out));
    }
  }
  NG_CUDA(cudaEventRecord(st->ev_out, st->copy_out));
  NG_CUDA(cudaStreamWaitEvent(s, st->ev_out, 0));
  NG_CUDA(cudaStreamSynchronize(s));
  return NGALORE_OK;
}

ngalore_status ngalore_poll_status(ngalore_state* st, int* per_matrix) {
  if (st == nullptr) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  NG_CUDA(cudaDeviceSynchronize());
  std::vector<int> h(st->n);
  NG_CUDA(cudaMemcpy(h.data(), st->d_status, sizeof(int) * st->n, cudaMemcpyDeviceToHost));
  Ctrl c{};
  NG_CUDA(cudaMemcpy(&c, st->d_ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost));
  NG_CUDA(cudaMemset(st->d_status, 0, sizeof(int) * st->n));
  // steps replayed from a CUDA graph advance only the device-side counters: take those over
  st->k = c.k;
  st->n_appended = c.n_appended;
  if (c.timeout_flag != 0) NG_CUDA(cudaMemset(&st->d_ctrl->timeout_flag, 0, sizeof(int)));
  ngalore_status first = NGALORE_OK;
  for (int i = 0; i < st->n; ++i) {
    if (per_matrix) per_matrix[i] = h[i];
    if (first == NGALORE_OK && h[i] != 0) first = static_cast<ngalore_status>(h[i]);
  }
  if (first == NGALORE_OK && c.timeout_flag != 0) first = NGALORE_ERR_TIMEOUT;
  return first;
}

ngalore_status ngalore_get_subspace(ngalore_state* st, int i, float* P, void* stream) {
  if (st == nullptr || i < 0 || i >= st->n || P == nullptr) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  const HostMat& hm = st->mats[i];
  NG_CUDA(cudaMemcpyAsync(P, st->h_desc[i].P32, sizeof(float) * hm.eM * hm.rp, cudaMemcpyDeviceToDevice,
                          static_cast<cudaStream_t>(stream)));
  return NGALORE_OK;
}

ngalore_status ngalore_get_working_subspace(ngalore_state* st, int i, float* P, void* stream) {
  if (st == nullptr || i < 0 || i >= st->n || P == nullptr) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  const HostMat& hm = st->mats[i];
  const long long cnt = static_cast<long long>(hm.eM) * hm.rp;
  widen_16_kernel<<<static_cast<unsigned>((cnt + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      st->h_desc[i].P16, P, cnt, hm.rp, st->h_desc[i].ldp, hm.right ? 0 : 1);
  st->launches += 1;
  NG_CUDA(cudaGetLastError());
  return NGALORE_OK;
}

ngalore_status ngalore_set_subspace(ngalore_state* st, int i, const float* P, void* stream) {
  if (st == nullptr || i < 0 || i >= st->n || P == nullptr) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  const HostMat& hm = st->mats[i];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  NG_CUDA(cudaMemcpyAsync(st->h_desc[i].P32, P, sizeof(float) * hm.eM * hm.rp, cudaMemcpyDeviceToDevice, s));
  ngalore_status rc = make_working_copies(st, i, s);
  if (rc != NGALORE_OK) return rc;
  st->subspace_set[i] = 1;
  st->has_subspace = true;  // stepping needs a projector for every matrix
  for (char c : st->subspace_set) st->has_subspace = st->has_subspace && c != 0;
  return NGALORE_OK;
}

ngalore_status ngalore_state_export(ngalore_state* st, void* blob, size_t* bytes) {
  if (st == nullptr || bytes == nullptr) return NGALORE_ERR_INVALID_ARG;
  const size_t need = sizeof(BlobHeader) + st->arena_bytes;
  if (blob == nullptr) { *bytes = need; return NGALORE_OK; }
  if (*bytes < need) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  NG_CUDA(cudaDeviceSynchronize());
  Ctrl c{};
  NG_CUDA(cudaMemcpy(&c, st->d_ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost));
  st->k = c.k;                      // the device-side counters are the authority (graph replays advance only them)
  st->n_appended = c.n_appended;
  BlobHeader h{};
  h.magic = kBlobMagic; h.arena_bytes = st->arena_bytes; h.k = st->k; h.n_appended = st->n_appended;
  h.n = st->n; h.r = st->r; h.s = st->s; h.has_subspace = st->has_subspace ? 1 : 0; h.shape_hash = st->shape_hash;
  std::memcpy(blob, &h, sizeof(h));
  NG_CUDA(cudaMemcpy(static_cast<char*>(blob) + sizeof(h), st->arena, st->arena_bytes, cudaMemcpyDeviceToHost));
  *bytes = need;
  return NGALORE_OK;
}

ngalore_status ngalore_state_import(ngalore_state* st, const void* blob, size_t bytes) {
  if (st == nullptr || blob == nullptr || bytes < sizeof(BlobHeader)) return NGALORE_ERR_INVALID_ARG;
  BlobHeader h{};
  std::memcpy(&h, blob, sizeof(h));
  if (h.magic != kBlobMagic || h.arena_bytes != st->arena_bytes || h.n != st->n || h.r != st->r || h.s != st->s ||
      h.shape_hash != st->shape_hash || bytes < sizeof(h) + h.arena_bytes)
    return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  NG_CUDA(cudaDeviceSynchronize());
  NG_CUDA(cudaMemcpy(st->arena, static_cast<const char*>(blob) + sizeof(h), st->arena_bytes, cudaMemcpyHostToDevice));
  // The blob brings back the step epoch of the exporting state.  The per-matrix flags of the stream kernel hold
  // epochs of steps this state ran before the import and could equal the next step's tag by accident (export, step,
  // import, step): clear them, together with the scheduling counters and anything a testing aid left behind.
  NG_CUDA(cudaMemset(st->d_flags, 0, sizeof(int) * 2 * st->n));
  Ctrl c{};
  NG_CUDA(cudaMemcpy(&c, st->d_ctrl, sizeof(Ctrl), cudaMemcpyDeviceToHost));
  c.timeout_flag = 0; c.work_counter = 0u; c.gemm_counter0 = 0u; c.gemm_counter1 = 0u;
  c.spin_limit = 0; c.debug_withhold = 0;
  NG_CUDA(cudaMemcpy(st->d_ctrl, &c, sizeof(Ctrl), cudaMemcpyHostToDevice));
  st->k = h.k; st->n_appended = h.n_appended; st->has_subspace = h.has_subspace != 0;
  st->subspace_set.assign(st->n, st->has_subspace ? 1 : 0);
  return NGALORE_OK;
}

ngalore_status ngalore_set_update_groups(ngalore_state* st, int n_groups) {
  if (st == nullptr || n_groups < 0 || n_groups > 4096) return NGALORE_ERR_INVALID_ARG;
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  NG_CUDA(cudaDeviceSynchronize());
  for (cudaEvent_t e : st->ev_upd) if (e) cudaEventDestroy(e);
  st->ev_upd.clear();
  st->upd_first.clear();
  if (n_groups <= 1) return NGALORE_OK;
  // contiguous groups of about equal weight traffic
  size_t total = 0;
  for (const HostMat& hm : st->mats) total += static_cast<size_t>(hm.M) * hm.N;
  const int want = n_groups < st->n ? n_groups : st->n;
  st->upd_first.assign(1, 0);
  size_t acc = 0;
  for (int i = 0; i < st->n; ++i) {
    acc += static_cast<size_t>(st->mats[i].M) * st->mats[i].N;
    const size_t done = st->upd_first.size();
    if (i + 1 < st->n && static_cast<int>(done) < want && acc * want >= total * done) st->upd_first.push_back(i + 1);
  }
  st->upd_first.push_back(st->n);
  st->ev_upd.assign(st->upd_first.size() - 1, nullptr);
  for (cudaEvent_t& e : st->ev_upd)
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) { e = nullptr; return NGALORE_ERR_CUDA; }
  return NGALORE_OK;
}

int ngalore_num_update_groups(const ngalore_state* st) {
  return st == nullptr ? 0 : (st->upd_first.size() > 1 ? static_cast<int>(st->upd_first.size()) - 1 : 1);
}

ngalore_status ngalore_update_group_range(const ngalore_state* st, int g, int* first, int* last) {
  if (st == nullptr || first == nullptr || last == nullptr || g < 0 || g >= ngalore_num_update_groups(st)) return NGALORE_ERR_INVALID_ARG;
  if (st->upd_first.size() > 1) { *first = st->upd_first[g]; *last = st->upd_first[g + 1]; }
  else { *first = 0; *last = st->n; }
  return NGALORE_OK;
}

ngalore_status ngalore_stream_wait_update(ngalore_state* st, int g, void* stream) {
  if (st == nullptr || g < 0 || g >= ngalore_num_update_groups(st)) return NGALORE_ERR_INVALID_ARG;
  if (st->upd_first.size() <= 1) return NGALORE_ERR_INVALID_ARG;   // no groups: order by the stepping stream itself
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  NG_CUDA(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), st->ev_upd[g], 0));
  return NGALORE_OK;
}

ngalore_status ngalore_debug_withhold_solution(ngalore_state* st, int matrix_index, int polls) {
  if (st == nullptr || matrix_index < 0 || matrix_index >= st->n || polls < 1 || polls > 1000000) return NGALORE_ERR_INVALID_ARG;
  if (st->s < 1 || st->opt.stream_impl == 1) return NGALORE_ERR_INVALID_ARG;
  if (!st->tc.gram_fused.empty() && st->tc.gram_fused[matrix_index]) return NGALORE_ERR_INVALID_ARG;
  if (st->sr.ready) return NGALORE_ERR_INVALID_ARG;   // the small-rank path has no wait to run out
  DeviceGuard guard(st->device);
  if (!guard.ok) return NGALORE_ERR_CUDA;
  NG_CUDA(cudaDeviceSynchronize());
  const int v[2] = {polls, matrix_index + 1};
  NG_CUDA(cudaMemcpy(&st->d_ctrl->spin_limit, v, sizeof(v), cudaMemcpyHostToDevice));
  return NGALORE_OK;
}

ngalore_status ngalore_set_lr(ngalore_state* st, double lr) {
  if (st == nullptr || !(lr == lr)) return NGALORE_ERR_INVALID_ARG;
  st->hyper.lr = static_cast<float>(lr);
  st->hyper_dirty = true;
  return NGALORE_OK;
}

int ngalore_num_matrices(const ngalore_state* st) { return st ? st->n : 0; }
int ngalore_rank(const ngalore_state* st, int i) { return (st && i >= 0 && i < st->n) ? st->mats[i].rp : -1; }
int ngalore_projects_right(const ngalore_state* st, int i) { return (st && i >= 0 && i < st->n) ? (st->mats[i].right ? 1 : 0) : -1; }
int ngalore_subspace_rows(const ngalore_state* st, int i) { return (st && i >= 0 && i < st->n) ? st->mats[i].eM : -1; }
int64_t ngalore_step_count(const ngalore_state* st) { return st ? st->k : -1; }
size_t ngalore_device_bytes(const ngalore_state* st) { return st ? st->arena_bytes + st->work_bytes + st->stage_bytes + st->tc.device_bytes + st->refresh.device_bytes + st->sr.device_bytes : 0; }
int64_t ngalore_launch_count(const ngalore_state* st) { return st ? st->launches : 0; }
int64_t ngalore_descriptor_uploads(const ngalore_state* st) { return st ? st->tc.bind_uploads : 0; }
int ngalore_uses_small_rank_path(const ngalore_state* st) { return (st && st->sr.ready) ? 1 : 0; }

ngalore_status ngalore_set_profiling(ngalore_state* st, int on) {
  if (st == nullptr) return NGALORE_ERR_INVALID_ARG;
  st->profiling = on != 0;
  st->ev_valid = false;
  return NGALORE_OK;
}

double ngalore_last_phase_ms(ngalore_state* st, int phase) {
  if (st == nullptr || phase < 0 || phase > 2 || !st->profiling || !st->ev_valid) return -1.0;
  DeviceGuard guard(st->device);
  if (cudaEventSynchronize(st->ev[3]) != cudaSuccess) return -1.0;
  float ms = 0.f;
  if (cudaEventElapsedTime(&ms, st->ev[phase], st->ev[phase + 1]) != cudaSuccess) return -1.0;
  return static_cast<double>(ms);
}

}  // extern "C"
