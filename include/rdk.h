/*
 * rdk.h -- C ABI of the B200 (sm_100a) library for the hot path of the Redistributing Drafter
 * Kernels (RDK) sampler of "Out-of-Vocabulary Sampling Boosts Speculative Decoding".
 *
 * For every row (one sequence at one draft position) the library
 *   1. soft-maxes the pruned drafter's n logits and projects them onto the intersection with the
 *      target vocabulary (Token-Level Intersection, Eq. "tli-drafter"; Algorithm 1 step 1) -> q',
 *   2. redistributes q' onto the full target vocabulary of N tokens, either exactly,
 *      w = M^T q' with a row-stochastic token-affinity matrix M (Algorithm 1 step 2, Eq.
 *      "symbolic-m"), or with the linear-time first-order formula
 *      theta = p^T q',  w_j = (N q'_j + theta p_j) / (N + p_j)   (Eq. "rdk-taylor"),
 *      and normalises q~ = w / S, S = sum_j w_j,
 *   3. draws a (possibly out-of-vocabulary) draft token d ~ q~, accepts it with probability
 *      min(1, p_d / q~_d) and otherwise draws a replacement from the normalised residual
 *      max(0, p - q~)   (Algorithm 1 step 3 = Algorithm 4 steps 4-8),
 *   4. reports the closed-form acceptance rate alpha = sum_j min(p_j, q~_j) (Definition 2.1).
 *
 * General rules
 *   - Every pointer is a DEVICE pointer unless its name ends in _host.  The library allocates no
 *     device memory and keeps no device state: inputs, outputs, the kept-id index, the affinity
 *     matrix and workspaces are caller-owned and are neither freed nor retained after a call.
 *     On the HOST the library keeps one small table per process: for every kept-id index that
 *     rdk_prepare_ids built, its address, (N, n) and whether the ids were ascending and valid.
 *     rdk_sample_and_verify consults it to pick a kernel; the entries are never removed (a few
 *     bytes each), and the kernels re-check the index header on the device, so an index buffer
 *     that was freed and reused for something else is detected, not trusted.
 *   - Calls enqueue work on the caller's cudaStream_t (passed as void*; NULL = default stream) and
 *     return at once; outputs are valid after the stream has been synchronised.  rdk_prepare_ids
 *     and rdk_sample_and_verify_host are the exceptions: they synchronise the stream themselves.
 *   - Every call returns an rdk_status.  Argument errors are detected on the host and launch
 *     nothing.  There is no CPU fallback: on a device that is not compute capability 10.x every
 *     compute call returns RDK_ERR_ARCH.
 *   - A row index is r = b * positions + pos; per-(row, trial) outputs are indexed r * trials + t.
 *   - Draws use the inverse CDF in ascending token id: the drawn token is the smallest j whose
 *     inclusive prefix sum exceeds u * total, u in [0, 1).  Uniform lane 0 drives the draft draw,
 *     lane 1 the acceptance test (accepted <=> u * q~_d < p_d), lane 2 the residual draw, lane 3
 *     is spare.
 */
#ifndef RDK_H_
#define RDK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum rdk_status {
    RDK_OK = 0,
    RDK_ERR_INVALID_ARG = 1,        /* null pointer, non-positive size, bad stride, bad enum      */
    RDK_ERR_BAD_IDS = 2,            /* two drafter indices map to one target token                */
    RDK_ERR_EMPTY_INTERSECTION = 3, /* no kept id lies in [0, N): the paper assumes I != {}       */
    RDK_ERR_UNSUPPORTED = 4,        /* valid request that this build does not implement           */
    RDK_ERR_WORKSPACE_TOO_SMALL = 5,
    RDK_ERR_ARCH = 6,               /* current device is not sm_100                               */
    RDK_ERR_CUDA = 7,               /* a CUDA call failed; text in rdk_last_error()               */
    RDK_ERR_TIMEOUT = 8             /* a bounded device-side wait expired (read from status_word) */
} rdk_status;

typedef enum rdk_dtype { RDK_F32 = 0, RDK_BF16 = 1 } rdk_dtype;
typedef enum rdk_kind { RDK_LOGITS = 0, RDK_PROBS = 1 } rdk_kind;
typedef enum rdk_mode { RDK_MODE_LINEAR = 0, RDK_MODE_PRECOMPUTED_W = 1 } rdk_mode;

/* rdk_problem.flags.  RDK_FLAG_ROW_KERNEL makes rdk_sample_and_verify take the one-CTA-per-row
 * kernel even where the streaming kernel would serve (the two can then be compared on the same
 * inputs; the row kernel divides exactly where the streaming kernel expands 1 / (N + p_j)).      */
#define RDK_FLAG_ROW_KERNEL 1
/* RDK_FLAG_W_AS_GIVEN (mode RDK_MODE_PRECOMPUTED_W only; RDK_ERR_INVALID_ARG elsewhere): q~ = w
 * itself instead of w / sum(w).  For a w whose entries are probabilities of a larger distribution
 * and sum to less than 1: the pruning-without-redistribution scheme of Sec. 5.2 ("Acceptance
 * recovery", scheme (a)), where the drafter's full-vocabulary q is masked to I and not
 * renormalised.  alpha, the rejection test and the residual max(0, p - w) then use w as it
 * stands; the draft token is still drawn in proportion to w (a draw needs a distribution); the S
 * output remains sum(w).  The caller guarantees 0 <= w_j and sum(w) <= 1.                         */
#define RDK_FLAG_W_AS_GIVEN 2

/* Which kernel a call of the linear mode takes (see rdk_sample_route).                           */
typedef enum rdk_route { RDK_ROUTE_ROW_KERNEL = 0, RDK_ROUTE_STREAM_KERNEL = 1 } rdk_route;

/* Physical layouts of the affinity matrix M (n rows i in I, N columns j in T).
 *   RDK_AFF_F32_ROWS : float  M[i * ld + j], ld >= N.           Contracted with fp32 FMAs.
 *   RDK_AFF_BF16_COLS: bf16  Mt[j * ld + i], ld >= n, ld % 8 == 0, base 16-byte aligned
 *                      (the transpose, so that the contraction index i is contiguous for both
 *                      operands).  Contracted on the tensor cores with fp32 accumulation.      */
typedef enum rdk_affinity_layout { RDK_AFF_F32_ROWS = 0, RDK_AFF_BF16_COLS = 1 } rdk_affinity_layout;

typedef struct rdk_problem {
    int32_t N;                  /* target vocabulary size |T|, >= 1                              */
    int32_t n;                  /* drafter entries per row, >= 1                                 */
    int32_t batch;              /* sequences                                                     */
    int32_t positions;          /* draft positions per sequence; rows = batch * positions        */
    int32_t target_dtype;       /* rdk_dtype of the target logits                                */
    int32_t drafter_dtype;      /* rdk_dtype of the drafter logits / probabilities               */
    int32_t drafter_kind;       /* rdk_kind: RDK_LOGITS are soft-maxed, RDK_PROBS taken as is    */
    int32_t flags;              /* 0, or an OR of RDK_FLAG_ROW_KERNEL, RDK_FLAG_W_AS_GIVEN       */
    int64_t target_row_stride;  /* elements between target rows; 0 means N                       */
    int64_t drafter_row_stride; /* elements between drafter rows; 0 means n                      */
    const void* kept_index;     /* device buffer filled by rdk_prepare_ids for this (N, n)       */
} rdk_problem;

typedef struct rdk_affinity {
    const void* data;           /* device; layout as rdk_affinity_layout says                    */
    int32_t layout;
    int32_t reserved;           /* must be 0                                                     */
    int64_t ld;                 /* leading dimension in elements                                 */
} rdk_affinity;

/* All members are device pointers, caller-allocated; any may be NULL (that output is skipped).  */
typedef struct rdk_outputs {
    int32_t* draft_token;       /* [rows * trials] d ~ q~ (may be outside the kept ids)          */
    int32_t* out_token;         /* [rows * trials] d if accepted, else the residual draw         */
    uint8_t* accepted;          /* [rows * trials] 1 / 0                                         */
    float*   accept_prob;       /* [rows * trials] min(1, p_d / q~_d)                            */
    float*   alpha;             /* [rows] sum_j min(p_j, q~_j)            (Definition 2.1)       */
    float*   theta;             /* [rows] p^T q'  (linear mode only)                             */
    float*   S;                 /* [rows] sum_j w_j                                              */
    float*   residual_mass;     /* [rows] sum_j max(0, p_j - q~_j) = 1 - alpha  (Lemma 2.3)      */
    int32_t* accepted_len;      /* [batch * trials] leading accepted positions (Alg. 4 step 7)   */
    int32_t* status_word;       /* [1] device-side error code, 0 when fine; caller zeroes it     */
} rdk_outputs;

/* ---------------------------------------------------------------------------------------------
 * Helpers
 * ------------------------------------------------------------------------------------------- */
int rdk_version(void);                          /* major * 1000 + minor                           */
const char* rdk_status_string(int status);      /* static string, never NULL                      */
const char* rdk_last_error(void);               /* thread-local detail of the last failure        */

/* ---------------------------------------------------------------------------------------------
 * Kept-id index.  The drafter's index i maps to target token kept_ids[i] (the intersection I of
 * Sec. 2; ids < 0 or >= N stand for drafter tokens outside the target vocabulary, the set F, and
 * are dropped by the TLI step).  rdk_prepare_ids validates the list and builds, in a caller-owned
 * device buffer of rdk_kept_index_bytes(N, n) bytes (256-byte aligned), a membership bitmask over
 * T with rank counts and the rank -> drafter-index table that the row kernels read, and, for
 * ascending valid ids and N >= 4096, the tables of the streaming kernel (which kept ids fall
 * into which segment of the vocabulary and where their target logits sit inside a CTA's slice,
 * for 2-byte and for 4-byte logits; about 4 n bytes + 80 KB).  Any order of ids is accepted;
 * ascending valid ids are the fastest case.
 *   kept_ids       device int32 [n]
 *   n_valid_host   host int*, may be NULL: receives the number of ids inside [0, N)
 * Synchronises `stream`.  Errors: RDK_ERR_BAD_IDS (duplicate id), RDK_ERR_EMPTY_INTERSECTION,
 * RDK_ERR_WORKSPACE_TOO_SMALL, RDK_ERR_INVALID_ARG.
 * ------------------------------------------------------------------------------------------- */
size_t rdk_kept_index_bytes(int32_t N, int32_t n);
int rdk_prepare_ids(const int32_t* kept_ids, int32_t n, int32_t N, void* kept_index,
                    size_t kept_index_bytes, int* n_valid_host, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_build_affinity -- Eq. "symbolic-m" (Sec. 4, "Token-affinity priors"), with the covariance
 * Omega replaced by the cosine similarity of token embeddings:
 *   Omega_ij = <e_{kappa_i}, e_j> / (|e_{kappa_i}| |e_j|),
 *   M_ij = exp(Omega_ij / tau) / sum_{k in T} exp(Omega_ik / tau),   i in I, j in T.
 * One-time preprocessing (the paper: "calculated once at preprocessing time").
 *   embeddings   device [N, d] of emb_dtype, row stride emb_row_stride elements (0 means d)
 *   kept_ids     device int32 [n]; rows whose id is outside [0, N) are written as zeros
 *   tau          > 0
 *   M_out        device, layout / ld as in rdk_affinity (data member is ignored; M_out is used)
 *   ws           device workspace of rdk_build_affinity_workspace_bytes(N, n, d) bytes
 * Arithmetic: fp32 dot products and soft-max; the result is rounded to bf16 (nearest even) only
 * when it is stored in the bf16 layout.  bf16 embeddings (d >= 64, 16-byte aligned rows) going to the
 * bf16 layout take the tensor cores for the dot products (bf16 products are exact, accumulation in
 * fp32), in chunks of 2048 kept rows through an fp32 scratch [N, 2048] inside the workspace; every
 * other combination uses fp32 FMAs.  Both routes compute the same quantity.  If a bounded wait
 * inside the tensor-core kernel expires (the call has no status word), element [0, 0] of M_out is
 * set to NaN.
 * ------------------------------------------------------------------------------------------- */
size_t rdk_build_affinity_workspace_bytes(int32_t N, int32_t n, int32_t d);
int rdk_build_affinity(const void* embeddings, int32_t emb_dtype, int32_t d, int64_t emb_row_stride,
                       const int32_t* kept_ids, int32_t n, int32_t N, float tau,
                       const rdk_affinity* M_desc, void* M_out, void* ws, size_t ws_bytes,
                       void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_redistribute_exact -- Algorithm 1 steps 1-2:  q' = TLI(softmax(drafter)),  w = M^T q'.
 *   drafter   device [rows, n] logits or probabilities (problem->drafter_kind / drafter_dtype)
 *   M         affinity matrix; RDK_AFF_BF16_COLS runs on the tensor cores (q' is rounded to bf16
 *             as the left operand, products accumulate in fp32), RDK_AFF_F32_ROWS uses fp32 FMAs
 *   w_out     device float [rows, N] (row stride N): un-normalised weights
 *   S_out     device float [rows] or NULL: S = sum_j w_j (q~ = w / S)
 *   ws        device workspace of rdk_exact_workspace_bytes(problem, M->layout) bytes, 256-byte
 *             aligned (holds the q' operand)
 *   status_word device int32 [1] or NULL: set to RDK_ERR_TIMEOUT if a bounded wait inside the
 *             tensor-core pipeline expires (the kernel then stops early and w_out is incomplete)
 * ------------------------------------------------------------------------------------------- */
size_t rdk_exact_workspace_bytes(const rdk_problem* problem, int32_t affinity_layout);
int rdk_redistribute_exact(const rdk_problem* problem, const void* drafter, const rdk_affinity* M,
                           float* w_out, float* S_out, void* ws, size_t ws_bytes,
                           int32_t* status_word, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_redistribute_exact_static -- the paper has no counterpart; this is a packaging variant of
 * rdk_redistribute_exact for callers that cannot allocate device memory: code running where
 * cudaMalloc is off limits (inside a stream capture, in a latency-critical serving loop that must
 * not touch the allocator, or in a host framework that owns all device memory and hands out only
 * input and output buffers).  Same arguments and results as rdk_redistribute_exact, minus the
 * workspace: the q' operand is staged in a fixed array of RDK_STATIC_SCRATCH_BYTES bytes that is
 * part of the library image (each GPU that loads the library carries it until the process exits).
 *   - Problems whose operand does not fit (rdk_exact_workspace_bytes(problem, layout) >
 *     RDK_STATIC_SCRATCH_BYTES) are refused with RDK_ERR_WORKSPACE_TOO_SMALL; nothing is launched.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress);
 *     make that first call outside any stream capture.  No call allocates or frees anything.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (the operand
 *     is rewritten in full by every call), but two calls whose kernels overlap on the GPU, e.g. on
 *     different streams, race on it: serialise them.
 * ------------------------------------------------------------------------------------------- */
#define RDK_STATIC_SCRATCH_BYTES (4u << 20)
int rdk_redistribute_exact_static(const rdk_problem* problem, const void* drafter,
                                  const rdk_affinity* M, float* w_out, float* S_out,
                                  int32_t* status_word, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_redistribute_linear -- Eq. "rdk-taylor" written out to memory (the element-wise checkable
 * form of the linear path; rdk_sample_and_verify never stores this N-long vector).
 *   target      device [rows, N] target logits (p = softmax(target))
 *   drafter     device [rows, n]
 *   qtilde_out  device float [rows, N] (row stride N): q~ = w / S
 *   theta_out   device float [rows] or NULL
 *   S_out       device float [rows] or NULL
 * ------------------------------------------------------------------------------------------- */
int rdk_redistribute_linear(const rdk_problem* problem, const void* target, const void* drafter,
                            float* qtilde_out, float* theta_out, float* S_out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_sample_and_verify -- Algorithm 1 step 3 / Algorithm 4 steps 4-8 for every row, fused with
 * the redistribution that feeds it.
 *   mode RDK_MODE_LINEAR:        q~ from Eq. "rdk-taylor", computed on the fly from target and
 *                                drafter (w is never stored); `w` must be NULL.
 *   mode RDK_MODE_PRECOMPUTED_W: q~ = w / sum(w) with w float [rows, N], row stride w_row_stride
 *                                elements (0 means N), e.g. from rdk_redistribute_exact;
 *                                `drafter` is ignored.
 *   target     device [rows, N] target logits
 *   uniforms   device float [rows, trials, 4] in [0, 1)
 *   trials     >= 1 independent draws per row (each uses its own 4 uniforms)
 *   out        see rdk_outputs
 *   ws         device workspace of rdk_sample_workspace_bytes(problem, mode, trials) bytes, 256-byte
 *              aligned (may be NULL when that size is 0).  The streaming kernels keep there one
 *              record of 4160 bytes per row (row scalars and per-segment sums of w, min(p, q~),
 *              max(0, p - q~), p), one 4-byte counter per (sequence, trial), and 64 bytes per
 *              (row, CTA sharing the row) through which those CTAs exchange their partial
 *              soft-max sums.  Its contents need no initialisation.  One workspace serves one call
 *              at a time: calls that share it must be ordered on one stream (they may be queued
 *              back to back without synchronising).  The call may be captured in a CUDA graph and
 *              the graph replayed: the second kernel wipes the exchanged records of a row once the
 *              row is drawn, so a replay never meets the previous replay's.
 * Kernels.  For N >= 4096 with ascending valid kept ids, 16-byte aligned target rows, a 16-byte
 * aligned drafter base and an even drafter row stride, the linear mode is TWO launches: a
 * persistent kernel (one CTA per SM; the first launch of a shape is a cooperative one, which proves
 * that the grid fits the SMs at hand) that streams every row from HBM once
 * and leaves the per-row record above, and a small kernel (one CTA per row and trial) that draws
 * the draft token, tests it and draws the replacement from those records, reading again only the
 * few 1024-token chunks the draws fall into.  There the quotient 1 / (N + p_j) is expanded in
 * x = p_j / N <= 2^-12 and terms of relative size x^2 (below 2^-24) are dropped.  Every other
 * problem takes the one-CTA-per-row kernel (three sweeps over the row, exact division), which is
 * several times slower; rdk_sample_route tells which one a call would take and why.  Both
 * streaming kernels are launched with programmatic stream serialisation: each may set itself up
 * while the previous kernel of the stream drains, but reads none of its inputs and touches nothing
 * of the workspace before that kernel is complete, so inputs written by the kernel queued just
 * before the call are safe.
 * If a bounded wait inside the kernel expires, out->status_word is set to RDK_ERR_TIMEOUT and the
 * outputs of that call are not valid.  Arithmetic of the linear mode: fp32.
 * ------------------------------------------------------------------------------------------- */
size_t rdk_sample_workspace_bytes(const rdk_problem* problem, int32_t mode, int32_t trials);
int rdk_sample_and_verify(const rdk_problem* problem, int32_t mode, const void* target,
                          const void* drafter, const float* w, int64_t w_row_stride,
                          const float* uniforms, int32_t trials, const rdk_outputs* out,
                          void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_sample_route -- host-only query (no CUDA call, nothing launched): which kernel
 * rdk_sample_and_verify would run Algorithm 4 steps 4-8 with for these arguments.  It sees what
 * rdk_stream_geometry cannot: the flags, alignment and strides of the rows, the workspace, and
 * whether the kept ids of problem->kept_index were ascending and valid when the index was built.
 *   why   host const char**, may be NULL: receives a static string naming the first reason the
 *         streaming kernel cannot serve ("" when it can)
 * Returns RDK_ROUTE_STREAM_KERNEL or RDK_ROUTE_ROW_KERNEL, or -(rdk_status) for a bad problem.
 * ------------------------------------------------------------------------------------------- */
int rdk_sample_route(const rdk_problem* problem, int32_t mode, const void* target,
                     const void* drafter, int32_t trials, const void* ws, size_t ws_bytes,
                     const char** why);

/* ---------------------------------------------------------------------------------------------
 * rdk_test_set_spin_limit -- for tests of the failure path only (the paper has no counterpart).
 * Every wait inside the streaming kernel (on a shared-memory barrier, on a record another CTA
 * publishes) gives up after a number of failed tries, records RDK_ERR_TIMEOUT in
 * out->status_word and lets the kernel run to its end.  This sets that number for later calls of
 * this process; 0 restores the default (2^17 tries of up to 2 us each).  With a limit of 1 the waits of an ordinary call
 * run out, which is how the tests reach the failure path without hanging or faulting anything.
 * ------------------------------------------------------------------------------------------- */
void rdk_test_set_spin_limit(uint32_t limit);

/* ---------------------------------------------------------------------------------------------
 * rdk_sample_and_verify_prior / rdk_redistribute_linear_prior -- the linear mode with a separate
 * prior: Eq. "rdk-taylor" uses p both as the direction of the affinity's principal component and
 * as the distribution to verify against; at draft time the true p is not known yet, so a caller
 * may supply the logits of a prior pi instead (theta = pi^T q', w_j = (N q'_j + theta pi_j) /
 * (N + pi_j), pi = softmax(prior)), while the rejection test, alpha and the residual use
 * p = softmax(target) as always.
 *   prior             device [rows, N] logits of the same dtype as the target, or one shared row
 *   prior_row_stride  elements between prior rows; 0 means one row shared by all rows
 * Everything else as in rdk_sample_and_verify (mode RDK_MODE_LINEAR) and rdk_redistribute_linear.
 * These calls take the one-CTA-per-row kernel and need no workspace.
 * ------------------------------------------------------------------------------------------- */
int rdk_sample_and_verify_prior(const rdk_problem* problem, const void* target, const void* prior,
                                int64_t prior_row_stride, const void* drafter, const float* uniforms,
                                int32_t trials, const rdk_outputs* out, void* stream);
int rdk_redistribute_linear_prior(const rdk_problem* problem, const void* target, const void* prior,
                                  int64_t prior_row_stride, const void* drafter, float* qtilde_out,
                                  float* theta_out, float* S_out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_stream_geometry -- host-only query (no CUDA call): how the streaming kernels of the linear
 * mode would lay a problem of N target tokens and n kept ids out, or supported = 0 when such a
 * problem takes the one-CTA-per-row kernel (N < 4096, or shapes beyond shared memory; unsorted
 * or invalid kept ids and unaligned rows also do, but are not known here).  A row is shared by
 * ctas_per_row CTAs of warps_per_cta streaming warps, each owning segment_tokens consecutive
 * tokens (Eq. "rdk-taylor" is evaluated per segment; ctas_per_row * warps_per_cta segments cover
 * the vocabulary); stages = depth of the shared-memory ring; live_rows - 1 = rows by which the
 * second visit of a row trails its first.  Returns RDK_OK, or RDK_ERR_INVALID_ARG.
 * ------------------------------------------------------------------------------------------- */
typedef struct rdk_stream_geometry_t {
    int32_t supported;
    int32_t ctas_per_row;
    int32_t warps_per_cta;
    int32_t segment_tokens;
    int32_t stages;
    int32_t live_rows;
    int32_t cached_slots_per_warp;
    int32_t reserved;
    int64_t dynamic_shared_bytes;
} rdk_stream_geometry_t;
int rdk_stream_geometry(int32_t N, int32_t n, int32_t target_dtype, int32_t drafter_dtype,
                        rdk_stream_geometry_t* out);


/* ---------------------------------------------------------------------------------------------
 * rdk_emit_sequences -- Algorithm 4 steps 7-9: what each sequence emits after verification.  For
 * sequence b and trial t, with j = number of leading accepted positions:
 *   seq_tokens[b, t, 0..j) = the accepted drafts d_1..d_j,
 *   seq_tokens[b, t, j]    = out_token of position j (the residual draw of the first rejection) if
 *                            j < positions, else a draw t ~ softmax(bonus_target[b]) -- the target
 *                            distribution after all drafts -- by inverse CDF with uniform lane 3 of
 *                            the sequence's last position,
 *   seq_len[b, t]          = j + 1  (between 1 and positions + 1).
 *   bonus_target  device [batch, N] target logits of problem->target_dtype, row stride in elements
 *                 (0 means N)
 *   uniforms, draft_token, accepted, out_token: as given to / produced by rdk_sample_and_verify
 *   seq_tokens    device int32 [batch, trials, positions + 1] (entries beyond seq_len are untouched)
 *   seq_len       device int32 [batch, trials]
 * Only problem->N, batch, positions and target_dtype are read.
 * ------------------------------------------------------------------------------------------- */
int rdk_emit_sequences(const rdk_problem* problem, const void* bonus_target, int64_t bonus_row_stride,
                       const float* uniforms, int32_t trials, const int32_t* draft_token,
                       const uint8_t* accepted, const int32_t* out_token, int32_t* seq_tokens,
                       int32_t* seq_len, void* stream);

/* ---------------------------------------------------------------------------------------------
 * rdk_sample_and_verify_host -- the same step (linear mode) for callers whose logits live in HOST
 * memory: copies target_host / drafter_host / uniforms_host to the caller's device staging
 * buffers, runs rdk_sample_and_verify, copies the per-(row, trial) and per-row results back and
 * synchronises the stream.  Host buffers should be pinned for full copy speed.
 *   problem->kept_index, staging buffers: device.   *_host: host.
 *   stage_target [rows * N], stage_drafter [rows * n] of the problem's dtypes, stage_uniforms
 *   float [rows * trials * 4], dev_out: device outputs as in rdk_outputs (members that are NULL
 *   are skipped, also in host_out); host_out: host arrays of the same shapes; ws as in
 *   rdk_sample_and_verify.
 * ------------------------------------------------------------------------------------------- */
int rdk_sample_and_verify_host(const rdk_problem* problem, const void* target_host,
                               const void* drafter_host, const float* uniforms_host,
                               int32_t trials, void* stage_target, void* stage_drafter,
                               float* stage_uniforms, const rdk_outputs* dev_out,
                               const rdk_outputs* host_out, void* ws, size_t ws_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RDK_H_ */
