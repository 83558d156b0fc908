/*
 * flop.h -- C ABI of the B200 (sm_100a) hot path of FLOP, factorized low-rank
 * pruning ("Structured Pruning of Large Language Models", arXiv 1910.04732).
 *
 * The layer is y = P G Q x with G = diag(z) (Section 4.1): W in R^{d_out x d_in}
 * is replaced by P in R^{d_out x r}, Q in R^{r x d_in} and one hard-concrete
 * gate z_k per rank-1 component p_k q_k (Section 3).
 *
 * Conventions for every entry point
 *   - Matrices are row-major with an element leading dimension (ld*).  Tokens
 *     are rows: X[T, d_in], Y[T, d_out], H'[T, r]; P[d_out, r]; Q[r, d_in].
 *   - Unless a parameter says HOST, every pointer is a DEVICE pointer owned by
 *     the caller.  The library allocates no device memory; scratch is passed
 *     in as (ws, ws_bytes) and sized with flop_workspace_bytes().  ws must be
 *     256-byte aligned.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*); no
 *     call synchronises unless it says so.
 *   - dt is the storage type of X, P, Q, Y, H' and of the activation
 *     gradients.  FLOP_BF16 computes on the tensor cores with fp32
 *     accumulation and needs every bf16 leading dimension to be a multiple of
 *     8 elements and every bf16 base pointer to be 16-byte aligned
 *     (FLOP_ERR_UNSUPPORTED otherwise).  FLOP_F32 computes in fp32 FMA.
 *   - Errors are return codes.  Arguments are checked on the host before
 *     anything is launched.  A device-side wait that runs out (a pipeline
 *     barrier that never completes) makes the kernel stop cleanly and record
 *     FLOP_ERR_TIMEOUT in a device status word read by flop_last_async_status().
 *   - The only environment variable the library reads is FLOP_DEBUG (1: print the failing CUDA call to
 *     stderr).  Variant switches for tuning exist only in a build with -DFLOP_TUNING (listed in flop_lib.cu).
 *   - Sizes of zero (T == 0, r == 0, k == 0, n == 0) are legal: outputs that
 *     exist are zero-filled where the mathematics says so, nothing else runs.
 */
#ifndef FLOP_H_
#define FLOP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FLOP_OK = 0,
  FLOP_ERR_INVALID_ARG = 1, /* null pointer, negative size, ld too small, bad enum; a bad device-side table */
  FLOP_ERR_UNSUPPORTED = 2, /* alignment / leading-dimension / size limit of the kernels   */
  FLOP_ERR_WORKSPACE = 3,   /* ws is NULL, misaligned or smaller than flop_workspace_bytes */
  FLOP_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed                           */
  FLOP_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up                          */
} flop_status_t;

typedef enum { FLOP_F32 = 0, FLOP_BF16 = 1 } flop_dtype_t;

/* Hard-concrete constants: temperature beta > 0 and stretch limits
 * gamma < 0 < 1 < zeta (the paper's l and r, Section 3; its formulas are the
 * beta = 1 case). */
typedef struct {
  float beta, gamma, zeta;
} flop_hc_params_t;

typedef enum {
  FLOP_OP_FWD = 0,         /* flop_gated_lowrank_fwd                   */
  FLOP_OP_BWD = 1,         /* flop_gated_lowrank_bwd                   */
  FLOP_OP_L0 = 2,          /* flop_expected_l0_lagrangian (T = gates n, r = n_seg) */
  FLOP_OP_COMPACT = 3,     /* flop_compact_ranks                       */
  FLOP_OP_COMPACT_FWD = 4, /* flop_compact_fwd (r = k)                 */
  FLOP_OP_EMBEDDING_BWD = 5 /* flop_gated_embedding_bwd (r = d_i)       */
} flop_op_t;

const char* flop_status_string(int status);

/* Synchronises `stream`, returns the device status word (FLOP_OK; FLOP_ERR_TIMEOUT when a bounded
 * device-side wait of an earlier call gave up; FLOP_ERR_INVALID_ARG when a kernel found a device-side
 * table it cannot use, see flop_expected_l0_lagrangian) and clears it.  flop_device_status is the same call
 * under its older name. */
int flop_last_async_status(void* stream);
int flop_device_status(void* stream);

/* Self-test of the bounded device-side wait (no counterpart in the paper): launches one thread that waits
 * on a barrier nothing will ever signal, for at most limit_cycles SM cycles (<= 2e9), then records
 * FLOP_ERR_TIMEOUT in the device status word and writes 1 to *gave_up_dev (DEVICE int).  The context stays
 * usable; flop_last_async_status() returns and clears the code. */
int flop_selftest_wait_timeout(int64_t limit_cycles, int* gave_up_dev, void* stream);

/* Instrumentation (no counterpart in the paper): kernels this library has launched so far in this
 * process.  Not synchronised with concurrent launches from other threads. */
unsigned long long flop_launch_count(void);

/* Host-only planning helper (no counterpart in the paper; no GPU needed): the static tile schedule a grouped
 * GEMM launch uses.  cost[n] (HOST) = cost of each work item in work-list order, units = persistent CTAs or CTA
 * pairs (1..148), n <= 2048.  Items are assigned by the longest-processing-time rule (sorted by cost, ties keep
 * list order, each to the least loaded unit, ties to the lower unit); when the round-robin deal is already within
 * 3 % of the lower bound max(mean load, longest item) it is kept.  unit_of_item[n] (HOST, nullable) receives
 * the unit of every item, *makespan the largest unit load, *rr_makespan the largest load of the round-robin deal
 * (item i to unit i % units) for comparison (both HOST, nullable).  FLOP_ERR_INVALID_ARG on bad sizes. */
int flop_plan_tile_schedule(const double* cost, int32_t n, int32_t units, int32_t* unit_of_item, double* makespan,
                            double* rr_makespan);

/* The queue of a chained launch (flop_gated_lowrank_*_chained; host only): stage[n] (HOST) is 0 for tiles that
 * wait for nothing and 1 for tiles that read a stage-0 output; key[n] (HOST) orders the tiles inside a stage (lower
 * first, ties keep list order).  queue_pos[n] (HOST, nullable) receives every item's position in the queue the
 * persistent CTA pairs draw from.  All stage-0 items come before all stage-1 items, which is what makes the
 * device-side waits free of cycles.  n <= 2048. */
int flop_plan_chain_queue(const int32_t* stage, const int64_t* key, int32_t n, int32_t* queue_pos);

/* Instrumentation (no counterpart in the paper).  While timing is on, every tensor-core GEMM launch is
 * bracketed by CUDA events on its stream; _end waits for them and returns the summed kernel time (ms), the
 * summed algorithmic flops 2 M N K of those launches and their number (HOST out pointers, nullable).
 * Single-threaded use only: the event list and the counters are not guarded against concurrent launches. */
int flop_gemm_timing_begin(void);
int flop_gemm_timing_end(double* total_ms, double* total_flops, int64_t* launches);

/* Device-side stamps (no counterpart in the paper): between _begin and _end, GEMM launch i is
 * issued with a pointer to stamps_dev[2i..2i+1] (DEVICE, zero-initialised by the caller) and writes
 * there the %globaltimer (ns) at which its first CTA passed the dependency wait and the latest
 * time at which one of its CTAs finished.  The pointers stay in the launches, so a CUDA graph
 * captured in between refreshes the stamps at every replay; this times kernels where host events
 * cannot be placed.  _end returns the number of stamped launches and the sum of their 2 M N K.
 * Single-threaded use only, like the event timing above. */
int flop_gemm_stamps_begin(unsigned long long* stamps_dev, int capacity);
int flop_gemm_stamps_end(int* launches, double* total_flops);
/* One small kernel on `stream`: acc_dev[0] += the sum of (end - start) over the `capacity` stamp pairs of stamps_dev
 * that have been written (unwritten pairs are zero), acc_dev[1] += 1 (DEVICE u64[2], zeroed by the caller).  Issued
 * at the end of a step that is captured in a CUDA graph, it adds up the GEMM kernel time of every replay on the
 * device, in the very replays that are being timed. */
int flop_gemm_stamps_accumulate(const unsigned long long* stamps_dev, int capacity, unsigned long long* acc_dev,
                                void* stream);

/* Bytes of scratch the given call needs (HOST out pointer).  For FLOP_OP_L0
 * pass the total number of gates as T and the number of segments as r. */
int flop_workspace_bytes(int op, int64_t T, int64_t d_in, int64_t d_out, int64_t r, int dt,
                         size_t* out_bytes);

/* The tensor-core GEMM every bf16 path is built from (Section 4.1: the layer is
 * "simple matrix multiplications"): D[M,N] = sum_k A(m,k) B(n,k), bf16 operands,
 * fp32 accumulation.  An operand is K-major (memory [MN rows, K cols],
 * *_mn_major = 0) or MN-major (memory [K rows, MN cols], *_mn_major = 1).
 * Supported pairs: (K,K) and (K,MN) store bf16 D (ld ldd), each column times the
 * optional col_scale[n]; (MN,MN) writes fp32 split-K slices
 * slices[s][m*ldN + n] with ldN = N rounded up to 4 and slice stride M*ldN, which
 * the caller adds up (the buffer must hold 32 slices unless splits is given).
 * bn (64, 128, 192, 256; 208 for a CTA pair with K-major B), cta2 (0: one CTA per 128-row tile; 1: a CTA pair per
 * 256-row tile) and splits fix the tile shape; bn = 0, cta2 = -1, splits = 0 leave
 * each choice to the library.  *n_slices_out (HOST, nullable) receives the number
 * of slices written (1 for a bf16 store). */
int flop_tc_gemm(const void* A, int64_t lda, int a_mn_major, const void* B, int64_t ldb,
                 int b_mn_major, void* D, int64_t ldd, const float* col_scale, float* slices,
                 int64_t M, int64_t N, int64_t K, int bn, int cta2, int splits, int* n_slices_out,
                 void* stream);

/* Gate sampling (Section 3, the inverse CDF G(u; alpha) of the hard-concrete
 * distribution), for gates j = 0..n-1:
 *     u_j   = ((x_j >> 9) + 1/2) 2^-23, x_j = word (j mod 4) of the Philox4x32-10
 *             block with counter (offset + j/4) and key `seed`
 *     s     = sigmoid((log u - log(1-u) + log_alpha) / beta)
 *     s_bar = s (zeta - gamma) + gamma,   z = min(1, max(0, s_bar))
 *     mask  = (z > 0),   dz_dla = dz/dlog_alpha (0 on the clamps)
 * Outputs z[n] f32, mask[n] u8 (nullable), dz_dla[n] f32 (nullable).  The
 * mask decision is taken in fp64 whenever fp32 could not decide it safely, so
 * it equals the fp64 evaluation of the formulas above. */
int flop_gate_sample(const float* log_alpha, int64_t n, flop_hc_params_t hc, uint64_t seed,
                     uint64_t offset, float* z, uint8_t* mask, float* dz_dla, void* stream);

/* The same sampler with the Philox counter offset taken from device memory:
 * gate j uses counter offset + *offset_dev + j/4 (Section 3 draws a fresh u for
 * every training batch).  A training step captured once in a CUDA graph keeps its
 * kernel arguments; with the offset on the device the caller advances it between
 * replays (any device-side add) and every replay draws a new mask. */
int flop_gate_sample_devoff(const float* log_alpha, int64_t n, flop_hc_params_t hc, uint64_t seed,
                            uint64_t offset, const uint64_t* offset_dev, float* z, uint8_t* mask,
                            float* dz_dla, void* stream);

/* Forward of the gated factorized layer (Section 4.1):
 *     H' = (X Q^T) * z   (column k times z_k, applied in the first GEMM's epilogue)
 *     Y  = H' P^T
 * H_save[T, r] (ld ldh) receives H' for the backward pass; it may be NULL
 * (inference), then H' lives in ws.  z is f32[r]. */
int flop_gated_lowrank_fwd(const void* X, int64_t ldx, const void* Q, int64_t ldq, const void* P,
                           int64_t ldp, const float* z, void* Y, int64_t ldy, void* H_save,
                           int64_t ldh, int64_t T, int64_t d_in, int64_t d_out, int64_t r, int dt,
                           void* ws, size_t ws_bytes, void* stream);

/* Backward (chain rule through Section 4.1's product; Section 3 notes that
 * theta and alpha both receive gradients):
 *     dH' = dY P            dP = dY^T H'          dQ = diag(z) (dH'^T X)
 *     dz_k = <Q[k,:], (dH'^T X)[k,:]>  (= sum_t H[t,k] dH'[t,k])
 *     dX  = dH' (diag(z) Q)                dlog_alpha = dz * dz_dla
 * H_save is the H' written by the forward call.  dX has type dt; dP, dQ have
 * type wgrad_dt; dlog_alpha is f32[r].  Any of dX, dP, dQ, dlog_alpha may be
 * NULL (skipped).  accumulate != 0 adds into dP, dQ and dlog_alpha instead of
 * overwriting them (dX is always overwritten). */
int flop_gated_lowrank_bwd(const void* dY, int64_t lddy, const void* X, int64_t ldx, const void* Q,
                           int64_t ldq, const void* P, int64_t ldp, const float* z,
                           const float* dz_dla, const void* H_save, int64_t ldh, void* dX,
                           int64_t lddx, void* dP, int64_t lddp, void* dQ, int64_t lddq,
                           float* dlog_alpha, int accumulate, int64_t T, int64_t d_in,
                           int64_t d_out, int64_t r, int dt, int wgrad_dt, void* ws,
                           size_t ws_bytes, void* stream);

/* Grouped forms: n independent problems (different weight matrices, e.g. the
 * Q/K/V projections that share an input, or all matrices of a layer whose weight
 * gradients are due together) run through the SAME sequence of kernels as n single
 * calls, but each GEMM stage is one persistent launch over the tiles of all problems,
 * so pipeline fill, epilogue drain and launch gaps are paid once per stage instead
 * of once per matrix (Section 4.1's products, batched).  Results match the single
 * calls within the storage-type tolerance (tile shapes and split-K factors may
 * differ).  `problems` is a HOST array; the pointers inside follow the conventions of
 * the single calls.  Forward: H_save is required (there is no scratch argument).
 * Backward: every problem brings its own workspace of at least
 * flop_workspace_bytes(FLOP_OP_BWD, ...) bytes; workspaces must not overlap. */
typedef struct {
  const void* X; int64_t ldx; const void* Q; int64_t ldq; const void* P; int64_t ldp;
  const float* z; void* Y; int64_t ldy; void* H_save; int64_t ldh;
  int64_t T, d_in, d_out, r;
  const int32_t* r_dev; /* nullable; see "Training on the active rank components" below */
} flop_fwd_problem_t;

typedef struct {
  const void* dY; int64_t lddy; const void* X; int64_t ldx; const void* Q; int64_t ldq;
  const void* P; int64_t ldp; const float* z; const float* dz_dla; const void* H_save; int64_t ldh;
  void* dX; int64_t lddx; void* dP; int64_t lddp; void* dQ; int64_t lddq; float* dlog_alpha;
  int64_t T, d_in, d_out, r;
  void* ws; size_t ws_bytes;
  const int32_t* r_dev; /* nullable */
  const void* Qz; int64_t ldqz; /* nullable: diag(z) Q formed beforehand by flop_scale_rows_grouped (same z, same Q) */
  int32_t defer_dlog_alpha;     /* != 0: leave the partial row dots of dlog_alpha in ws; flop_dlog_alpha_finish_grouped adds them up */
} flop_bwd_problem_t;

/* diag(z) Q for n matrices in one launch: Qz[k, :] = z[k] * Q[k, :] (r x d_in, bf16, rounded once).  The
 * backward pass multiplies by it (dX = dH' (diag(z) Q), chain rule on Section 4.1); it depends only on the gate
 * sample and the weights, so a training step may form it once, right after flop_gate_sample, for all
 * matrices of the model, and pass it to the grouped / chained backward calls (flop_bwd_problem_t.Qz).
 * Problems that leave Qz NULL have it formed inside the backward call, in their workspace.  HOST array. */
typedef struct {
  const void* Q; int64_t ldq; const float* z; void* Qz; int64_t ldqz; int64_t r, d_in;
} flop_scale_rows_t;
int flop_scale_rows_grouped(const flop_scale_rows_t* problems, int n, int dt, void* stream);

/* Second stage of dlog_alpha for n problems in one launch (Section 3: alpha receives gradients with theta).  The
 * grouped / chained backward calls fuse dz_k = <Q[k,:], (dH'^T X)[k,:]> into the dQ product as partial row dots;
 * adding the partials and multiplying by dz_dla is a small second stage.  A problem with defer_dlog_alpha != 0
 * leaves its partials in its workspace instead; this call then writes dlog_alpha (=|+= with accumulate) for every
 * problem given, in fixed summation order.  Pass the same problem structs (ws, sizes, dz_dla, dlog_alpha) as to the
 * backward calls, any number of them together (e.g. all matrices of a model once per step); a workspace must not be
 * reused by another backward call in between.  bf16 only.  HOST array. */
int flop_dlog_alpha_finish_grouped(const flop_bwd_problem_t* problems, int n, int accumulate, int dt, void* stream);

int flop_gated_lowrank_fwd_grouped(const flop_fwd_problem_t* problems, int n, int dt, void* stream);
int flop_gated_lowrank_bwd_grouped(const flop_bwd_problem_t* problems, int n, int accumulate, int dt,
                                   int wgrad_dt, void* stream);

/* Chained forms: the same results as the grouped calls, with the dependent products of the call in ONE
 * persistent launch (Section 4.1: y = P G Q x is two products that feed each other; its chain rule is two
 * products, dH' = dY P and dP, followed by two that read dH').  The tiles of H' = (X Q^T) * z and of
 * Y = H' P^T share one work list; a tile of the second product waits, on the device, for the 256-row block
 * of H' it reads (counters in `sync`), instead of the whole first launch draining before the second fills.
 * The backward call likewise runs {dH', dP} and {dX, dQ} in one launch, forms diag(z) Q inside it and
 * finishes dlog_alpha inside it (no small kernels before or after).
 *   sync       DEVICE, 16-byte aligned, at least flop_sync_bytes() bytes.  The CALLER zero-fills it once
 *              (e.g. cudaMemsetAsync) before its first use; every call leaves it zero-filled again, also
 *              inside a replayed CUDA graph.  Calls that share a sync area must be ordered on the GPU
 *              (same stream, or events); concurrent calls need separate areas.  If a call ever reports
 *              FLOP_ERR_TIMEOUT through flop_last_async_status(), zero-fill the area again.
 *   Fallback   When the shapes do not allow one launch (fp32 storage, a product that needs split-K or
 *              one-CTA tiles, more than 24 products, more counters than the area holds) the call runs the
 *              grouped sequence of launches; results are the same.
 *   Every wait on a counter is bounded like the pipeline waits (FLOP_ERR_TIMEOUT in the status word).
 * flop_sync_bytes: HOST out pointer. */
int flop_sync_bytes(size_t* out_bytes);
int flop_gated_lowrank_fwd_chained(const flop_fwd_problem_t* problems, int n, int dt, void* sync,
                                   size_t sync_bytes, void* stream);
int flop_gated_lowrank_bwd_chained(const flop_bwd_problem_t* problems, int n, int accumulate, int dt,
                                   int wgrad_dt, void* sync, size_t sync_bytes, void* stream);

/* Training on the active rank components only (Section 4.3, last paragraph: the
 * mask is shared by the batch, so "parameters that are only active for the current
 * batch" are selected and the matrix products run on smaller matrices).
 *
 * flop_active_ranks_gather, per problem: idx = {k : z_k > 0} ascending, pos = its
 * inverse (-1 for closed gates), *k_dev = their number, z_c = z[idx],
 * dz_dla_c = dz_dla[idx] (both zero beyond k), Q_c[c,:] = Q[idx[c],:] (NOT scaled by
 * the gate), P_c[:,c] = P[:,idx[c]]; rows of Q_c / columns of P_c from k up to the
 * next multiple of 64 are zero.  Qz_c (nullable, leading dimension ldqzc) receives
 * diag(z_c) Q_c in the same launch, rounded to bf16 as flop_scale_rows_grouped rounds
 * it: the buffer a backward problem takes as Qz.  All compact buffers have the
 * capacity of the full rank r.  bf16 only.
 *
 * The grouped forward/backward calls then take the compact buffers in place of
 * P, Q, z, dz_dla, H_save, dP, dQ, dlog_alpha, with r = the capacity and
 * r_dev = k_dev: the effective rank is read on the device, GEMM tiles beyond it are
 * skipped and K loops stop at the 64-block holding component k-1.  Entries of the
 * outputs beyond k are unspecified.  Y and dX are the full results.
 *
 * flop_active_ranks_scatter writes the full gradients: dP[:,idx] = dP_c,
 * dQ[idx,:] = dQ_c, dlog_alpha[idx] = dlog_alpha_c and exact zeros elsewhere
 * (accumulate != 0: += instead).  Any of the three outputs may be NULL. */
typedef struct {
  const float* z; const float* dz_dla; const void* P; int64_t ldp; const void* Q; int64_t ldq;
  int64_t d_in, d_out, r;
  int32_t* idx; int32_t* pos; int32_t* k_dev; float* z_c; float* dz_dla_c;
  void* P_c; int64_t ldpc; void* Q_c; int64_t ldqc;
  void* Qz_c; int64_t ldqzc;
} flop_active_gather_t;

typedef struct {
  const int32_t* idx; const int32_t* pos; const int32_t* k_dev; int64_t d_in, d_out, r;
  const void* dP_c; int64_t lddpc; const void* dQ_c; int64_t lddqc; const float* dlog_alpha_c;
  void* dP; int64_t lddp; void* dQ; int64_t lddq; float* dlog_alpha;
} flop_active_scatter_t;

int flop_active_ranks_gather(const flop_active_gather_t* problems, int n, int dt, void* stream);
int flop_active_ranks_scatter(const flop_active_scatter_t* problems, int n, int accumulate, int wgrad_dt,
                              void* stream);

/* Expected size and augmented-Lagrangian penalty over all gates of all
 * matrices at once (Eq. 3 and Section 4.3).  Segment i (one weight matrix)
 * owns gates seg_off[i]..seg_off[i+1]-1 of log_alpha; each of its gates
 * stands for seg_size[i] = d_in + d_out parameters.
 *     pi_j = sigmoid(log_alpha_j - beta log(-gamma/zeta))
 *     s = sum_j pi_j size_j / sum_j size_j,   g = lambda1 (s - t) + lambda2 (s - t)^2
 * out4 = {s, g, dg/dlambda1, dg/dlambda2}; seg_expected[n_seg] (nullable) =
 * sum of pi_j per segment; dlog_alpha[n] (nullable) += dg/dlog_alpha.
 * n is the total number of gates.  seg_off[n_seg + 1] (DEVICE) must partition
 * [0, n): seg_off[0] = 0, ascending, seg_off[n_seg] = n.  The table is in device
 * memory, so it is checked on the device: a table that breaks this rule makes the
 * call write NaN to out4, leave everything else untouched and record
 * FLOP_ERR_INVALID_ARG in the status word flop_last_async_status() returns.
 * target[1] and lambda[2] are DEVICE pointers so that an optimiser can update
 * them on the device.  n_seg <= 4096. */
int flop_expected_l0_lagrangian(const float* log_alpha, int64_t n, const int64_t* seg_off,
                                const float* seg_size, int32_t n_seg, flop_hc_params_t hc,
                                const float* target, const float* lambda, float* out4,
                                float* seg_expected, float* dlog_alpha, void* ws, size_t ws_bytes,
                                void* stream);

/* The same computation as flop_expected_l0_lagrangian for callers that cannot
 * allocate device memory at all (the paper has no counterpart; this is a
 * deployment convenience).  Such callers exist: code running inside someone
 * else's memory plan -- an inference server or training loop whose pool was
 * sized up front and is now frozen, a plug-in that is handed tensors but no
 * allocator, a region where cudaMalloc would synchronise the device or is
 * simply forbidden.  The caller passes only inputs and outputs; the kernels'
 * scratch is a fixed array that is part of the loaded library (about 35 KB,
 * held on every GPU that loads the library until the process exits), so the
 * call performs no cudaMalloc/cudaFree and uses no allocating library routine.
 *   - Limits: n <= 1,048,576 gates and n_seg <= 4096 segments; larger sizes
 *     return FLOP_ERR_UNSUPPORTED (FLOP_DEBUG=1 prints the limits) and must use
 *     flop_expected_l0_lagrangian with a caller-provided workspace.
 *   - The first call on each device looks up the device address of the
 *     built-in array (with that device current); make that first call outside
 *     any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the
 *     previous call left in it.  Nothing in it has to start at zero (every
 *     value read is rewritten by the same call first), but two calls whose
 *     kernels overlap on the GPU -- different streams, no ordering between
 *     them -- race on it: order them. */
int flop_expected_l0_lagrangian_noalloc(const float* log_alpha, int64_t n, const int64_t* seg_off,
                                        const float* seg_size, int32_t n_seg, flop_hc_params_t hc,
                                        const float* target, const float* lambda, float* out4,
                                        float* seg_expected, float* dlog_alpha, void* stream);

/* Gated adaptive embedding of one word cluster (Section 4.2): E~ = E G O with E[n_rows, d_i] the
 * reduced-dimension embeddings of the cluster's words, O[d_i, d] the projection to the model
 * dimension and G = diag(z) pruning the d_i reduced dimensions.  ids[T] (int32, DEVICE) are row
 * indices into E (values outside [0, n_rows) are clamped).  bf16 only.
 *   forward : H_save[T, d_i] = E[ids, :] * z (required, it feeds the backward pass), Y[T, d] = H_save O
 *   backward: dH' = dY O^T, dO = H_save^T dY (type wgrad_dt; overwritten or += with accumulate),
 *             dE[ids[t], :] += dH'[t, :] * z  (fp32, ALWAYS accumulated with atomic adds because words
 *             repeat across tokens: clear dE before the first call of a step; the order of the adds
 *             is not fixed, so dE is reproducible only to fp32 rounding),
 *             dlog_alpha = dz_dla * sum_t E[ids[t], :] dH'[t, :]  (fixed summation order).
 *   Any of dE, dO, dlog_alpha may be NULL.  dO is written in place with 16-byte stores: its pointer must be
 *   16-byte aligned and lddo a multiple of 8 (bf16) or 4 (fp32) elements, else FLOP_ERR_UNSUPPORTED (checked
 *   before anything is launched).  Workspace: flop_workspace_bytes(FLOP_OP_EMBEDDING_BWD, T,
 *   0, 0, d_i, dt).  The tied softmax side of the same cluster, logits = ((h O^T) * z) E^T, is
 *   flop_gated_lowrank_fwd/bwd with Q = O^T and P = E. */
int flop_gated_embedding_fwd(const int32_t* ids, int64_t T, const void* E, int64_t lde, int64_t n_rows,
                             const void* O, int64_t ldo, const float* z, void* Y, int64_t ldy, void* H_save,
                             int64_t ldh, int64_t d_i, int64_t d, int dt, void* stream);
int flop_gated_embedding_bwd(const void* dY, int64_t lddy, const int32_t* ids, int64_t T, const void* E,
                             int64_t lde, int64_t n_rows, const void* O, int64_t ldo, const float* z,
                             const float* dz_dla, const void* H_save, int64_t ldh, float* dE, int64_t ldde,
                             void* dO, int64_t lddo, float* dlog_alpha, int accumulate, int64_t d_i, int64_t d,
                             int dt, int wgrad_dt, void* ws, size_t ws_bytes, void* stream);

/* FLOP-AGP variant (Section 5, baselines): magnitude-based pruning of the learnable diagonal mask
 * G = diag(g) instead of hard-concrete gates.  Segment i (one weight matrix) owns
 * g[seg_off[i]..seg_off[i+1]): its round(sparsity * r_i) entries of smallest |g| are pruned (ties at the
 * cut keep the lower indices); z = g on kept entries and 0 elsewhere, mask = [kept] (nullable),
 * dz_dg = [kept] (nullable), seg_l1[i] = sum |g| over the segment (nullable; the L1 term on the masks
 * is l1 times their sum), dg (nullable) += l1 * sign(g).  sparsity[1] is a DEVICE scalar so that a
 * schedule can advance it on the device.  The forward/backward calls then take z and dz_dg where they
 * take the sampled gate and dz_dla; the dlog_alpha they return is the gradient with respect to g. */
int flop_agp_gates(const float* g, int64_t n, const int64_t* seg_off, int32_t n_seg, const float* sparsity,
                   float l1, float* z, uint8_t* mask, float* dz_dg, float* seg_l1, float* dg, void* stream);

/* Deterministic gates and compaction of one weight matrix (Sections 4.4, 4.1).
 * mode 0: log_alpha_or_z holds log_alpha; k = floor(sum_j pi_j + 1/2); the k
 *         gates with the largest log_alpha are kept (ties: lower index) with
 *         value pi_j, the rest are 0.
 * mode 1: log_alpha_or_z holds a gate vector z; component j is kept iff z_j > 0.
 * Writes idx[r] (first k entries valid, ascending), k_dev[1], z_det[r]
 * (nullable) and, when P/Q/Pc/Qc are given (all or none),
 *     Pc[d_out, k] = P[:, idx]          (ld ldpc >= max k the caller allows, e.g. r)
 *     Qc[k, d_in]  = diag(z[idx]) Q[idx, :]   (the gate is absorbed into Q)
 * Columns >= k of Pc and rows >= k of Qc are left untouched.  r <= 65536. */
int flop_compact_ranks(const float* log_alpha_or_z, int mode, flop_hc_params_t hc, int64_t r,
                       const void* P, int64_t ldp, const void* Q, int64_t ldq, int64_t d_in,
                       int64_t d_out, int dt, int32_t* idx, int32_t* k_dev, float* z_det, void* Pc,
                       int64_t ldpc, void* Qc, int64_t ldqc, void* ws, size_t ws_bytes,
                       void* stream);

/* Inference forward on compact factors (Section 4.1: "simple matrix
 * multiplications"): Y = (X Qc^T) Pc^T with k surviving components, k known
 * on the host (read k_dev once after flop_compact_ranks). */
int flop_compact_fwd(const void* X, int64_t ldx, const void* Qc, int64_t ldqc, const void* Pc,
                     int64_t ldpc, void* Y, int64_t ldy, int64_t T, int64_t d_in, int64_t d_out,
                     int64_t k, int dt, void* ws, size_t ws_bytes, void* stream);

/* On-chip forward chain (Section 4.1: y = P G Q x as two products): Y = ((X Q^T) * z) P^T in ONE launch; the
 * rank-r intermediate is accumulated in tensor memory, gated, rounded to bf16 and handed to the second product
 * through shared memory, so it never reaches global memory (nothing is saved for a backward pass: this is an
 * inference call).  z is f32[r] or NULL (compact factors from flop_compact_ranks carry the gate in Qc already:
 * pass Qc, Pc, k as Q, P, r).  bf16 only, r <= 512 (FLOP_ERR_UNSUPPORTED beyond; use flop_compact_fwd /
 * flop_gated_lowrank_fwd, which choose between this kernel and two launches by shape).  Needs no workspace.
 * Results equal the two-launch path's up to fp32 summation order. */
int flop_chain_fwd(const void* X, int64_t ldx, const void* Q, int64_t ldq, const void* P, int64_t ldp,
                   const float* z, void* Y, int64_t ldy, int64_t T, int64_t d_in, int64_t d_out, int64_t r,
                   int dt, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FLOP_H_ */
