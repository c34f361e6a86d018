/*
 * ngalore.h -- C ABI of the Natural GaLore optimizer step for NVIDIA B200 (sm_100a).
 *
 * One ngalore_state owns, on the current CUDA device, the optimizer state of a
 * set of 2-D weight matrices.  For a matrix W (rows x cols = M x N, row-major,
 * fp32) with gradient G (M x N, row-major, bf16) one step computes
 *
 *   R  = P^T G                                   low-rank projection        (Sec. 1, "GaLore" paragraph)
 *   H[head] <- R, ring of the s latest R         stacked gradient matrix    (Sec. 2.4)
 *   K_ij = <H_i, H_j> / c                        empirical Fisher, mean of outer products (Sec. 2.2)
 *   (lambda I + K) w = e_cur, by Cholesky        the s x s system           (Sec. 2.4; equals S z = y after scaling)
 *   N~ = sum_i w_i H_i                           natural gradient F^-1 R    (Sec. 2.4, Woodbury identity)
 *   m, v, u = m / sqrt(v + eps)                  Adam moments as printed    (Sec. 2.2)
 *   W <- (1 - lr wd) W - lr P u                  update with decoupled decay (Sec. 2.2 update equation; AdamW)
 *
 * and, every T steps, first refreshes P to an orthonormal basis of the
 * dominant r'-dimensional left singular subspace of G, r' = min(r, M, N)
 * (Sec. 1: P from the compact SVD of the gradient, "updated periodically").
 * With ngalore_options.projection_rule = 1 a matrix with M >= N uses the mirrored
 * form instead: R = G Q, W <- (1 - lr wd) W - lr u Q^T, Q (N x r') from the
 * right singular vectors; everything between projection and update is the same.
 *
 * Conventions
 *  - All matrix pointers are DEVICE pointers unless a parameter says "host".
 *    Arrays of pointers (W, G below) are HOST arrays of device pointers.
 *  - W and G are dense row-major with leading dimension cols; cols must be a
 *    multiple of 8 and every pointer 16-byte aligned.  The caller owns W and G;
 *    the library owns everything else and frees it in ngalore_destroy.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    ngalore_step and ngalore_refresh_subspace enqueue work and return; they do
 *    not synchronise and do not allocate.
 *  - Host-detectable errors are returned at once and leave the state untouched.
 *    Errors found on the device set a per-matrix status word that
 *    ngalore_poll_status reports.  A non-finite gradient or a non-positive
 *    Cholesky pivot leaves that matrix's W, m and v unchanged for the step (its
 *    gradient enters the history as zero).  Every wait inside a kernel is
 *    bounded; when the wait for a matrix's solved weights runs out, that
 *    matrix's W is left unchanged for the step and its status is
 *    NGALORE_ERR_TIMEOUT (parts of its m and v may already have advanced); when
 *    a wait inside a GEMM pipeline runs out, the kernel stops issuing work and
 *    ngalore_poll_status returns NGALORE_ERR_TIMEOUT for the state as a whole:
 *    restore it from a checkpoint.  No call traps, aborts or spins for ever.
 *  - A state is bound to the device that was current in ngalore_create and is
 *    not safe for concurrent calls from several threads.
 */
#ifndef NGALORE_H
#define NGALORE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ngalore_state ngalore_state;

typedef struct {
  int64_t rows; /* M */
  int64_t cols; /* N, multiple of 8 */
} ngalore_shape;

typedef enum {
  NGALORE_OK = 0,
  NGALORE_ERR_INVALID_ARG = 1,
  NGALORE_ERR_ALLOC = 2,
  NGALORE_ERR_CUDA = 3,
  NGALORE_ERR_UNSUPPORTED_DEVICE = 4, /* the device is not compute capability 10.x */
  NGALORE_ERR_NO_SUBSPACE = 5,        /* step before any refresh / set_subspace with T == 0 */
  NGALORE_ERR_NOT_SPD = 6,            /* device: Cholesky pivot <= 0 */
  NGALORE_ERR_NONFINITE = 7,          /* device: NaN or Inf reached the Gram matrix */
  NGALORE_ERR_TIMEOUT = 8             /* device: a bounded wait inside a kernel ran out */
} ngalore_status;

/* Optional settings; pass NULL to ngalore_create for the defaults shown. */
typedef struct {
  int32_t struct_size;              /* = sizeof(ngalore_options) */
  int32_t gemm_impl;                /* 0 (default): tensor-core (tcgen05) projection GEMMs; 1: plain SIMT GEMMs (debug) */
  int32_t power_iterations;         /* subspace-iteration sweeps in the refresh; <= 0 selects the default 6 */
  int32_t reset_history_on_refresh; /* default 0: history, m and v survive a refresh */
  uint64_t seed;                    /* seed of the refresh's random test matrix and of the stochastic rounding of
                                       moments_bf16; 0 selects a fixed default (0x9E3779B97F4A7C15) */
  int32_t stream_impl;              /* 0 (default): fused Gram/solve/moment kernel; 1: separate plain kernels (debug) */
  int32_t projection_rule;          /* 0 (default): every matrix is projected on the left, R = P^T G, as the paper
                                       writes it; 1: the short-side rule of GaLore, which the paper's "most steps are
                                       similar to GaLore" (start of Sec. 2.4) inherits: a matrix with rows >= cols is
                                       projected on the right, R = G Q (rows x r'), W <- (1 - lr wd) W - lr u Q^T, with
                                       Q (cols x r') spanning the leading right singular vectors of G */
  int32_t history_bf16;             /* 0 (default): the ring of low-rank gradients is fp32.  1: reduced-precision state
                                       (the paper's conclusion names it as future work): the gradient of the current
                                       step takes part in fp32, which the Woodbury form needs, and is stored as bf16
                                       afterwards; the Gram matrix is kept that of the stored values.  Halves the
                                       history traffic and memory.  Needs s >= 1 and the fused stream kernel. */
  int32_t gram_fusion;              /* 0 (default): the new Gram row comes from the Gram tiles of the stream kernel.
                                       1: where the workload allows it (rank-512 class shapes, left projection, K of
                                       at most 8192, fp32 history of at most 16 slots, rows and columns multiples of
                                       32) it is formed in the epilogue of the projection GEMM instead, so that the
                                       first read of the history runs under the tensor-core work; same results to
                                       rounding.  Not faster than the default as built, hence off unless asked for. */
  int32_t ritz_columns;             /* the eigensolve at the end of a refresh rotates the leading ritz_columns
                                       columns of the refreshed basis into Ritz vectors (approximate singular
                                       vectors, in falling order of their singular value) within their own span; the
                                       remaining columns complete an orthonormal basis of the subspace as the
                                       subspace iteration left them.  0 (default): 256 (at most about a hundred
                                       singular values can be separated from both neighbours by 1e-2 sigma_1, and the
                                       iteration orders its basis by strength, so the determined singular vectors sit
                                       at the front; a weak one close to the noise level is still spread over a few
                                       hundred columns of an unconverged basis, which is why the default is not
                                       smaller); -1: all r' columns (the full Rayleigh-Ritz step; the cost of the
                                       eigensolve grows with the cube of the number of columns). */
  int32_t moments_bf16;             /* 0 (default): the Adam moments are fp32.  1: reduced-precision state (the paper's
                                       conclusion names it as future work): m is stored as bf16 rounded to nearest; v is
                                       stored as bf16 with stochastic rounding (one step changes v by a relative
                                       1 - beta2, less than half a bf16 unit, so rounding to nearest would freeze it),
                                       its random bits from Philox-4x32-10 keyed by `seed` with the counter (element
                                       index / 4, matrix index, step index).  The direction of a step comes from the
                                       unrounded moments.  Halves the moments' memory and traffic.  Needs the fused
                                       stream kernel and the left projection. */
  int32_t small_rank_path;          /* 0 (default): the tensor-core kernels at every rank.  1: when every matrix has
                                       r' <= 8 (the fine-tuning ranks 4 and 8 of Sec. 4.2 and 4.3), the projection is
                                       on the left, history and moments are fp32 and s <= 16, the step runs as two
                                       kernels without tensor cores that touch every element of G and W once with
                                       plain loads and stores (projection + Gram row; solve + moments + weight
                                       update).  Same results to rounding.  Measured slower than the default as built
                                       (strips of 64 columns stream G and W in pieces too short for the memory
                                       system), hence off unless asked for.  The path is left when update groups
                                       are set. */
} ngalore_options;

/*
 * Create the state for n_matrices weight matrices (Sec. 2.2-2.4 name the
 * hyper-parameters: rank r, history length s, refresh period T, Tikhonov
 * lambda, learning rate, Adam betas and eps, weight decay).
 *   shapes      host array of n_matrices shapes (at most 65535 matrices per state)
 *   r >= 1      target rank; per matrix r' = min(r, rows, cols); r' may not exceed 875 (the orthonormalisation
 *               of the refresh keeps 32 rows of r' doubles in shared memory), else NGALORE_ERR_INVALID_ARG
 *   s in [0,32] history length; 0 disables the Fisher term (plain GaLore)
 *   T >= 0      refresh period in steps; 0 = never refresh automatically
 *   lambda > 0 when s > 0
 * Moments and history start at zero / empty; P is unset until the first
 * refresh or ngalore_set_subspace.  Allocates all device memory the state will
 * ever need (cudaMalloc) on the current device.
 */
ngalore_status ngalore_create(const ngalore_shape* shapes, int n_matrices, int r, int s, int T,
                              double lambda, double lr, double beta1, double beta2, double eps,
                              double wd, const ngalore_options* opt, ngalore_state** out);

/* Free the state and all its device memory (synchronises the device). NULL is allowed. */
void ngalore_destroy(ngalore_state* st);

/*
 * One optimizer step over every matrix (equations at the top of this file).
 *   W  host array of n_matrices device pointers, fp32 M x N, updated in place
 *   G  host array of n_matrices device pointers, bf16 bit patterns M x N, read only
 * If T > 0 and the step index k satisfies k mod T == 0, the subspace of every
 * matrix is refreshed from G first.  Increments k.
 * The TMA descriptors of W and G are cached per array of pointers (at most 32 arrays, fewer for very many
 * matrices; the least recently used is overwritten): the first call with a given pair of arrays encodes and
 * uploads them, a later call with the same pointers enqueues kernels only (no copies), so it can be captured in a
 * CUDA graph.  Such a graph stays valid until its array of pointers has been pushed out of that cache.  A call
 * under stream capture leaves the host-side step counter alone and a replay advances the device-side ring
 * position and step index only, so the automatic refresh (which the host decides) cannot follow replays: create
 * the state with T = 0 when replaying from a graph and call ngalore_refresh_subspace yourself.
 */
ngalore_status ngalore_step(ngalore_state* st, float* const* W, const uint16_t* const* G, void* stream);

/*
 * Refresh P from G without stepping (Sec. 1: P spans the leading left singular
 * vectors of the gradient).  matrix_index = -1 refreshes all matrices, else one
 * (G is still the full array of n_matrices pointers; only entry matrix_index is read).
 * Uses a randomized subspace iteration; P is orthonormal to fp32 accuracy and is
 * stored both as an fp32 master and as the working copies the step reads (the master's values rounded to bf16).
 * Degenerate gradients: a gradient of zeros (a frozen layer) has no leading subspace; its matrix gets the first r'
 * unit vectors as P and no status.  A gradient with entries that are not finite gets the same P and
 * NGALORE_ERR_NONFINITE in its status word; the other matrices are refreshed as usual.
 */
ngalore_status ngalore_refresh_subspace(ngalore_state* st, const uint16_t* const* G, int matrix_index,
                                        void* stream);

/*
 * Same step with HOST buffers: copies W and G to internal device staging,
 * steps, copies W back and waits.  W_host / G_host are host arrays of HOST
 * pointers (pinned memory gives asynchronous copies).  Needs staging memory of
 * the size of all W and G, allocated on first use, together with two internal
 * copy streams: G goes in first, the projection and the history phase run while
 * W is still arriving, and W moves in groups of matrices whose copy in,
 * back-projection and copy out overlap across groups.  The work is ordered
 * after what `stream` holds at the call, and the call returns when all of it
 * is complete.
 */
ngalore_status ngalore_step_host(ngalore_state* st, float* const* W_host, const uint16_t* const* G_host,
                                 void* stream);

/* Wait for the state's work and copy the per-matrix status words (ngalore_status values)
 * to the host array `per_matrix` (n_matrices ints; may be NULL); clears them on the device.
 * Returns NGALORE_OK when all are OK, else the first non-OK status. */
ngalore_status ngalore_poll_status(ngalore_state* st, int* per_matrix);

/* Copy the fp32 master of the projector of matrix i (ngalore_subspace_rows(i) x r', row-major: P, or Q for a
 * matrix projected on the right) to / from the device buffer P.
 * set also rebuilds the working copies; the step uses the values rounded to bf16. */
ngalore_status ngalore_get_subspace(ngalore_state* st, int i, float* P, void* stream);
ngalore_status ngalore_set_subspace(ngalore_state* st, int i, const float* P, void* stream);
/* Copy the working copy of the projector (its bf16-rounded values, widened to fp32, same shape) to the device buffer P. */
ngalore_status ngalore_get_working_subspace(ngalore_state* st, int i, float* P, void* stream);

/* Checkpoint: with blob == NULL stores the needed size in *bytes; else copies the whole state
 * (P, m, v, history, Gram matrices, counters) into the HOST buffer blob (synchronises).
 * import restores it into a state created with identical shapes and r, s. */
ngalore_status ngalore_state_export(ngalore_state* st, void* blob, size_t* bytes);
ngalore_status ngalore_state_import(ngalore_state* st, const void* blob, size_t bytes);

/*
 * Update groups (the paper's related work: optimizer-state sharding, where ranks exchange updated weights; also any
 * consumer that wants the weights of the first layers before the last ones are done).  With n_groups >= 2 the
 * back-projection + weight update of ngalore_step runs as n_groups launches over contiguous ranges of matrices of
 * about equal size, and an event is recorded on the stepping stream after each.  ngalore_update_group_range gives
 * the matrices [first, last) of group g; ngalore_stream_wait_update makes `stream` wait until the latest enqueued
 * step has updated group g, so work on that stream (a copy, a collective, a forward pass) overlaps the update of
 * the later groups.  n_groups <= 1 restores the single launch.  Synchronises the device; not meant for steps
 * replayed from a CUDA graph (the events belong to the live stream).
 */
ngalore_status ngalore_set_update_groups(ngalore_state* st, int n_groups);
int ngalore_num_update_groups(const ngalore_state* st);
ngalore_status ngalore_update_group_range(const ngalore_state* st, int g, int* first, int* last);
ngalore_status ngalore_stream_wait_update(ngalore_state* st, int g, void* stream);

/*
 * Testing aid (no counterpart in the paper): in the next ngalore_step only, the solved weights of matrix
 * `matrix_index` are computed but not announced, and the tiles that wait for them give up after `polls` polls
 * (1 .. 1000000, about 100 ns each) instead of the default limit.  The step then ends normally with
 * NGALORE_ERR_TIMEOUT in that matrix's status word and its W unchanged; the following step is a regular one.
 * This is how the tests exercise a bounded wait that runs out; nothing hangs or traps.  Synchronises the device.
 * Not available with s = 0, stream_impl = 1, or for a matrix whose Gram row is formed by gram_fusion.
 */
ngalore_status ngalore_debug_withhold_solution(ngalore_state* st, int matrix_index, int polls);

/* Change the learning rate used from the next step on. */
ngalore_status ngalore_set_lr(ngalore_state* st, double lr);

/* Introspection (host values, no device work). */
int ngalore_num_matrices(const ngalore_state* st);
int ngalore_rank(const ngalore_state* st, int i);          /* r' of matrix i, -1 if i is out of range */
int ngalore_projects_right(const ngalore_state* st, int i); /* 1 if matrix i is projected on the right, 0 if on the left, -1 if out of range */
int ngalore_subspace_rows(const ngalore_state* st, int i);  /* rows of its projector: M (left) or N (right), -1 if out of range */
int64_t ngalore_step_count(const ngalore_state* st);        /* k as the host last knew it: steps replayed from a CUDA
                                                               graph are counted on the device and taken over by
                                                               ngalore_poll_status and ngalore_state_export */
size_t ngalore_device_bytes(const ngalore_state* st);       /* device memory held by the state */
/* Kernels launched by the library on behalf of this state since creation. */
int64_t ngalore_launch_count(const ngalore_state* st);
int ngalore_uses_small_rank_path(const ngalore_state* st);  /* 1 if the state takes the small-rank path (see options) */
/* How many times ngalore_step had to encode and upload the TMA descriptors of a (W, G) pair of pointer arrays
 * (see ngalore_step: once per distinct pair while it stays cached). */
int64_t ngalore_descriptor_uploads(const ngalore_state* st);

/* Per-phase timing of ngalore_step with CUDA events recorded on the launching stream.
 * phase: 0 projection GEMM (R = P^T G), 1 Gram / solve / moment kernels, 2 back-projection + W update.
 * ngalore_last_phase_ms waits for the step and returns milliseconds, or a negative value when
 * profiling is off or no step has run. */
ngalore_status ngalore_set_profiling(ngalore_state* st, int on);
double ngalore_last_phase_ms(ngalore_state* st, int phase);

/*
 * Natural-gradient transform of one matrix without any allocation.  (The paper has no counterpart:
 * this entry point exists for callers that cannot obtain device memory themselves -- code running
 * under a fixed, pre-carved memory budget, inside another framework's allocator-free region, or in
 * a process where cudaMalloc is forbidden after start-up -- and therefore cannot use ngalore_create.)
 *
 * Given the ring H of low-rank gradients (s slots of n fp32 elements each, slot-major, `count` of them
 * valid, the newest in slot `cur`) and the caller-kept raw Gram matrix K (s x s doubles, K_ij = <H_i, H_j>,
 * zero before the first call), it refreshes row and column `cur` of K, solves
 * (lambda I + K / count) w = e_cur by Cholesky in fp64 and writes out = sum_j w_j H_j (n floats).
 * This equals F^-1 applied to the newest gradient with F = lambda I + (1/count) sum_j vec(H_j) vec(H_j)^T,
 * the same arithmetic ngalore_step performs per matrix.
 *
 * All pointers are device pointers owned by the caller; H and out 16-byte aligned; n a multiple of 4.
 * `status` (device int, may be NULL) receives NGALORE_ERR_NOT_SPD / NGALORE_ERR_NONFINITE when the solve
 * fails (out is then all zeros); it is only ever set, so zero it beforehand.
 *
 * Scratch: the per-tile partial sums and the weights live in a 256.5 KiB array that is part of the
 * library image on every GPU that loads it, which bounds n at 8,388,608 elements per slot; larger n is
 * rejected with NGALORE_ERR_INVALID_ARG.  The call uses no cudaMalloc/cudaFree and no allocating library
 * routine.  The first call on a device looks up the array's device address; make that first call outside
 * any stream capture.  All calls on a device share the array (it keeps the previous call's contents, all
 * of which the next call overwrites before reading): two calls whose kernels may overlap on the GPU race,
 * so issue them on one stream or order them with events.  Asynchronous on `stream`.
 */
ngalore_status ngalore_natural_gradient_static(const float* H, int64_t n, int s, int count, int cur, double lambda,
                                               double* K, float* out, int* status, void* stream);

const char* ngalore_status_string(ngalore_status s);

#ifdef __cplusplus
}
#endif
#endif /* NGALORE_H */
