/*
 * entmax_attn.h -- C ABI of the fused alpha-entmax / ASEntmax attention library for NVIDIA B200
 * (sm_100a).  Plain pointers and sizes only; no framework types.
 *
 * What the library computes (notation of the paper; row i = query, column j = key):
 *
 *   n_i   = number of keys row i attends to: i+1 under the causal mask j <= i (Sec. 2.1, the sum
 *           over j <= i), N otherwise; with n_mode = 1, N for every row.
 *   c_i   = delta_h + beta_h * (ln n_i)^gamma_h     ASEntmax scale of head h (Eq. "asentmax");
 *           c_i = delta_h when n_i = 1; c_i = 1 when beta/gamma/delta are all NULL.
 *   s_ij  = c_i * <q_i, k_j> * sm_scale             attention logits (Sec. 2.1, z_ij = <q_i,k_j>/sqrt(d))
 *   tau_i : sum_j [(alpha-1) s_ij - tau_i]_+^(1/(alpha-1)) = 1          (Eq. 1, threshold)
 *   p_ij  = [(alpha-1) s_ij - tau_i]_+^(1/(alpha-1))                    (Eq. 1); exactly 0 when
 *           (alpha-1) s_ij <= tau_i (App. A)
 *   O_i   = sum_j p_ij v_j                                              (Sec. 2.1)
 *
 * Backward (Jacobian of Eq. 1 by implicit differentiation):
 *   dP_ij = <dO_i, v_j>,  u_ij = p_ij^(2-alpha) on the support and 0 off it,
 *   dS_ij = u_ij * (dP_ij - sum_l u_il dP_il / sum_l u_il),
 *   dQ_i = c_i sm_scale sum_j dS_ij k_j,  dK_j = sum_i c_i sm_scale dS_ij q_i,  dV_j = sum_i p_ij dO_i.
 *
 * General conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller.  The library allocates no device
 *     memory, never synchronises the device or a stream, and enqueues all work in the order of
 *     `cuda_stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).  The backward
 *     calls clear their accumulators on a stream of the library's own that is forked from and joined
 *     back to `cuda_stream` with events inside the call: the caller sees plain stream order.
 *   - Q, K, V, O, dO, dQ, dK, dV share one layout: [batch, heads, seq, head_dim] with head_dim
 *     innermost and contiguous; the other three strides come from the params struct (in elements).
 *     tau is [batch, heads, seq] float32, contiguous.  beta, gamma, delta are [heads] float32.
 *   - All tensor pointers must be 16-byte aligned and all strides multiples of 8 elements.
 *   - Functions return ENTMAX_ATTN_OK (0) or a negative entmax_attn_status.  On a validation error
 *     (every code except ENTMAX_ATTN_ECUDA) nothing has been enqueued; after ENTMAX_ATTN_ECUDA some of the
 *     call's work may already be on the stream and the outputs are undefined
 *     (entmax_attn_last_cuda_error() gives the CUDA error, for every entry point).  Device-side conditions
 *     are reported through `device_status`.
 *   - Non-finite values in Q, K, V or dO give unspecified results (never a fault).
 *   - alpha > 2 (the paper's retrieval experiments use 4 ... 64): the exponent 1/(alpha-1) is below 1, p is not
 *     Lipschitz at the edge of the support and u = p^(2-alpha) is unbounded there.  The thresholds come from a
 *     bracketed iteration (App. A's bisection bracket with Newton steps inside) instead of Newton from the left.
 *     Results are as accurate as float32 allows: a key that sits d above the threshold weighs d^(1/(alpha-1)), so the
 *     spacing of tau in float32 (about 4e-6 at |tau| = 50) caps the accuracy of P at about 2e-3 for alpha = 3 and
 *     2e-2 for alpha = 4; far beyond that only rows that are one-hot or exact ties come out exact, and the backward
 *     pass of a row with a key within 1e-3 of its threshold is unspecified (finite).
 *   - Sequences of different lengths in one batch: pad them on the right.  Under the causal mask a valid
 *     row never sees a padded key, so no extra mask is needed; give the padded rows dO = 0 and their
 *     content cannot reach dK, dV either (their own O, tau, dQ rows are to be ignored).  Non-causal
 *     problems have no padding mask.
 */
#ifndef ENTMAX_ATTN_H_
#define ENTMAX_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ENTMAX_ATTN_DTYPE_BF16 0 /* Q,K,V,dO in, O,dQ,dK,dV out: bfloat16; scores on tcgen05 tensor cores */
#define ENTMAX_ATTN_DTYPE_FP32 1 /* everything float32; scores by fp32 FMA (meets the tighter fp32 tolerance) */

typedef enum {
  ENTMAX_ATTN_OK = 0,
  ENTMAX_ATTN_EINVAL_SHAPE = -1,     /* batch/heads/seq < 1, head_dim not 64 or 128, bad strides, too many rows */
  ENTMAX_ATTN_EINVAL_ALPHA = -2,     /* alpha not in (1, 64] or not finite; sm_scale not finite or negative    */
  ENTMAX_ATTN_EINVAL_DTYPE = -3,     /* dtype is neither ENTMAX_ATTN_DTYPE_BF16 nor ENTMAX_ATTN_DTYPE_FP32      */
  ENTMAX_ATTN_EINVAL_ALIGN = -4,     /* a tensor pointer is not 16-byte aligned                                 */
  ENTMAX_ATTN_EINVAL_WORKSPACE = -5, /* workspace NULL, misaligned (256 B) or smaller than workspace_bytes()    */
  ENTMAX_ATTN_EINVAL_NULL = -6,      /* a required pointer is NULL, or only some of beta/gamma/delta are given  */
  ENTMAX_ATTN_ECUDA = -7,            /* a CUDA call failed; see entmax_attn_last_cuda_error()                   */
  ENTMAX_ATTN_EUNSUPPORTED = -8,     /* the device is not sm_100 (bf16 path needs tcgen05/TMA)                  */
  ENTMAX_ATTN_ETOOLARGE = -9         /* entmax_attn_fwd_static: the problem does not fit the built-in scratch  */
} entmax_attn_status;

typedef struct {
  int32_t batch, heads, seq, head_dim; /* head_dim in {64, 128}; seq >= 1, any value (tails are predicated)      */
  int32_t dtype;                       /* ENTMAX_ATTN_DTYPE_*                                                    */
  int32_t causal;                      /* 0 / 1; causal keeps j <= i, diagonal included                          */
  int32_t n_mode;                      /* 0: n_i = keys visible to row i; 1: n_i = seq for every row             */
  float alpha;                         /* 1 < alpha <= 64; 1.25, 1.5 and 2 use multiplication-only powers; beyond 2
                                          see "alpha > 2" below                                                   */
  float sm_scale;                      /* 0 means 1/sqrt(head_dim)                                               */
  int64_t stride_b, stride_h, stride_n; /* elements; all 0 means contiguous [batch, heads, seq, head_dim]        */
} entmax_attn_params;

/* Words of the optional device status array (int32[ENTMAX_ATTN_STATUS_WORDS], device memory, written
 * by the kernels of a call; zeroed at the start of that call). */
#define ENTMAX_ATTN_STATUS_WORDS 8
#define ENTMAX_ATTN_STATUS_FLAGS 0         /* bit field below; 0 = clean run                                   */
#define ENTMAX_ATTN_STATUS_DENSE_ROWS 1    /* rows whose support did not fit the sparse list (dense fallback)  */
#define ENTMAX_ATTN_STATUS_TILE_SWEEPS 2   /* forward: full-length sweeps over K spent by the dense-tile path, summed over tiles */
#define ENTMAX_ATTN_STATUS_TILES 3         /* 128-row Q tiles the dense-tile path of this call processed           */
#define ENTMAX_ATTN_STATUS_SKIPPED_STEPS 4 /* ALiBi heads: (256-row item, 256-key tile) steps of the score sweep that
                                              the hard-cutoff window left out ...                                 */
#define ENTMAX_ATTN_STATUS_SCORED_STEPS 5  /* ... and steps it still scored (both 0 without ALiBi slopes)          */
#define ENTMAX_ATTN_FLAG_WAIT_EXPIRED 1    /* a bounded on-chip wait ran out; outputs of that call are invalid */
#define ENTMAX_ATTN_FLAG_BAD_SCALE 2       /* some c_i was not finite                                          */
#define ENTMAX_ATTN_FLAG_BAD_LENGTH 4      /* entmax_attn_decode_fwd: some kv_len[b] outside [q_len, kv_capacity] */

/* Bytes of scratch the caller must pass to entmax_attn_fwd (is_bwd = 0) or entmax_attn_bwd
 * (is_bwd = 1) for these params.  Returns 0 if the params are invalid.  No paper counterpart: the
 * paper does not discuss memory. */
size_t entmax_attn_workspace_bytes(const entmax_attn_params* params, int is_bwd);

/* Forward pass: Eq. 1 applied to the ASEntmax-scaled logits of every query row (Eq. "asentmax",
 * Sec. 2.1), output O and the per-row threshold tau.
 *   q, k, v      in,  device, layout above, dtype per params->dtype
 *   beta, gamma, delta   in, device float32[heads]; pass all three or none (none: c_i = 1)
 *   o            out, device, same layout/dtype as q
 *   tau          out, device float32 [batch, heads, seq]; Eq. 1's tau (a one-hot row has
 *                tau = (alpha-1) s_max - 1)
 *   workspace    device scratch, 256-byte aligned, >= entmax_attn_workspace_bytes(params, 0); contents
 *                on return: see entmax_attn_workspace_layout
 *   device_status  optional device int32[ENTMAX_ATTN_STATUS_WORDS]
 * Errors: negative status (see the general conventions). */
int entmax_attn_fwd(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                    const float* beta, const float* gamma, const float* delta, void* o, float* tau,
                    void* workspace, size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

/* Backward pass: the Jacobian of Eq. 1 (see the top of this file) and the three input gradients.
 *   tau          in, device float32 [batch, heads, seq]: the thresholds the forward call returned
 *   d_o          in, gradient w.r.t. O, layout/dtype of q
 *   dq, dk, dv   out, layout/dtype of q (overwritten, not accumulated into)
 *   workspace    >= entmax_attn_workspace_bytes(params, 1)
 * No other state of the forward call is needed. */
int entmax_attn_bwd(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                    const float* beta, const float* gamma, const float* delta, const float* tau,
                    const void* d_o, void* dq, void* dk, void* dv, void* workspace,
                    size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

/* Backward pass that also returns the gradients of the ASEntmax scale (Eq. "asentmax": the temperature
 * c_i = delta_h + beta_h (log n_i)^gamma_h is learnable).  By the chain rule through s_ij = c_i z_ij,
 * z_ij = <q_i,k_j> sm_scale:
 *   d_scale_rows[b,h,i] = dL/dc_i = sum_j dS_ij z_ij            out, device float32 [batch,heads,seq] or NULL
 *   ddelta[h] = sum_{b,i} dL/dc_i,  dbeta[h] = sum_{b,i: n_i>1} dL/dc_i (log n_i)^gamma_h,
 *   dgamma[h] = sum_{b,i: n_i>1} dL/dc_i beta_h (log n_i)^gamma_h log(log n_i)
 *                                                               out, device float32 [heads]; all three or none;
 *                                                               they need beta, gamma, delta to be given
 * d_scale_rows is what a caller with per-query scales (its own c_i table) differentiates further.
 * Everything else as entmax_attn_bwd, which is this call with the four extra outputs NULL. */
int entmax_attn_bwd_scale(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                          const float* beta, const float* gamma, const float* delta, const float* tau,
                          const void* d_o, void* dq, void* dk, void* dv, float* d_scale_rows, float* dbeta,
                          float* dgamma, float* ddelta, void* workspace, size_t workspace_bytes,
                          int32_t* device_status, void* cuda_stream);

/* Forward / backward with a per-query scale table instead of per-head beta, gamma, delta: the paper's
 * full ASEntmax makes beta and gamma functions of the query (Sec. 4.1: beta = softplus(X w_beta),
 * gamma = s tanh(X w_gamma)), so c_i differs per batch element.  The caller evaluates Eq. "asentmax"
 * upstream and passes
 *   c_rows        in, device float32 [batch, heads, seq]: c_i of every query row (any finite value)
 * and gets back, from the backward call,
 *   d_scale_rows  out, device float32 [batch, heads, seq] or NULL: dL/dc_i, to be chained into its own
 *                 projection weights.
 * params->n_mode is ignored; everything else as entmax_attn_fwd / entmax_attn_bwd. */
int entmax_attn_fwd_rowscale(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                             const float* c_rows, void* o, float* tau, void* workspace, size_t workspace_bytes,
                             int32_t* device_status, void* cuda_stream);
int entmax_attn_bwd_rowscale(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                             const float* c_rows, const float* tau, const void* d_o, void* dq, void* dk, void* dv,
                             float* d_scale_rows, void* workspace, size_t workspace_bytes, int32_t* device_status,
                             void* cuda_stream);

/* The content-dependent scale itself (Sec. 4.1): for query token i of batch element b and head h
 *   beta = softplus(<x_bi, w_beta_h>),  gamma = gamma_range * tanh(<x_bi, w_gamma_h>),
 *   c = delta_h + beta (log n_i)^gamma        (Eq. "asentmax"; c = delta_h when n_i = 1),
 * n_i = i + 1 when causal and n_mode = 0, seq otherwise.  The forward call writes the table that
 * entmax_attn_fwd_rowscale / entmax_attn_bwd_rowscale take; the backward call takes the d_scale_rows those return and
 * applies the chain rule: dL/dw_beta, dL/dw_gamma [heads, d_model], dL/ddelta [heads] and dL/dx (the part of it that
 * flows through the scale; the caller adds it to the gradient x gets from its other uses).
 *   x            in,  device [batch, seq, d_model] contiguous, x_dtype (ENTMAX_ATTN_DTYPE_*)
 *   w_beta, w_gamma   in, device float32 [heads, d_model]; delta in, device float32 [heads]
 *   c_rows       out, device float32 [batch, heads, seq]
 *   d_scale_rows in,  device float32 [batch, heads, seq]
 *   dw_beta, dw_gamma out, device float32 [heads, d_model] (overwritten); ddelta out, float32 [heads] or NULL;
 *   dx           out, device [batch, seq, d_model] in x_dtype (overwritten) or NULL
 * heads <= 64.  Errors as for the other entry points (gamma_range must be positive and finite: EINVAL_ALPHA). */
typedef struct {
  int32_t batch, heads, seq, d_model;
  int32_t x_dtype;
  int32_t causal, n_mode;
  float gamma_range;
} entmax_attn_proj_params;
int entmax_attn_scale_proj_fwd(const entmax_attn_proj_params* params, const void* x, const float* w_beta,
                               const float* w_gamma, const float* delta, float* c_rows, void* cuda_stream);
int entmax_attn_scale_proj_bwd(const entmax_attn_proj_params* params, const void* x, const float* w_beta,
                               const float* w_gamma, const float* d_scale_rows, float* dw_beta, float* dw_gamma,
                               float* ddelta, void* dx, void* cuda_stream);

/* Extended forward / backward: every optional input and output of the calls above in one struct, plus the
 * ALiBi positional term of the paper's NAPE scheme (App. B: half of the heads add m_h (j - i) to the
 * logits z_ij = <q_i,k_j> sm_scale, j <= i; the other half use slope 0).  The ASEntmax scale multiplies
 * the whole logit, bias included (Eq. "asentmax" scales the logit vector).
 *   c_rows        in,  [batch, heads, seq] per-query scales; excludes beta, gamma, delta
 *   alibi_slopes  in,  [heads] slopes m_h >= 0 (0 = no positional term for that head); float32 problems
 *                 apply -m_h |i - j| on both sides of the query, bfloat16 problems need causal = 1
 *                 (ENTMAX_ATTN_EUNSUPPORTED otherwise)
 *   d_scale_rows, dbeta, dgamma, ddelta   out (backward only), as in entmax_attn_bwd_scale
 *   fwd_workspace saved state of the forward call, see the member below
 * Any member may be NULL; extras itself may be NULL.  Slopes get no gradient (the paper keeps them fixed). */
typedef struct {
  const float* c_rows;
  const float* alibi_slopes;
  float* d_scale_rows;
  float* dbeta;
  float* dgamma;
  float* ddelta;
  const void* fwd_workspace; /* backward only, bfloat16 problems: the workspace of the forward call on the same
                                inputs, untouched since it returned.  It still holds the support of every row, so
                                the backward pass skips its own score sweep (which otherwise recomputes Q K^T to
                                find the support from tau).  Must not be the buffer passed as `workspace`.        */
  const void* saved_supports; /* backward only, bfloat16 problems: the compact copy entmax_attn_save_supports made
                                of the forward call's supports (takes precedence over fwd_workspace).              */
} entmax_attn_extras;
/* Compact saved state for the backward pass.  Keeping the whole forward workspace alive until the backward
 * pass costs about 2 KB per query row; the supports themselves are a few entries per row.  This call copies,
 * for every row, its support size and up to ENTMAX_ATTN_SAVED_SLOTS support entries out of a finished forward
 * call's workspace into `saved` (entmax_attn_saved_bytes(params) bytes, 256-byte aligned: 4 + 8 *
 * ENTMAX_ATTN_SAVED_SLOTS bytes per row).  Passed as extras.saved_supports, it lets the backward pass skip its
 * score sweep like fwd_workspace does; rows whose support has more entries than the slots, and rows the
 * dense-tile path computed, are recomputed on the tensor cores instead.  bfloat16 problems only.  (The paper
 * has no counterpart: it does not discuss what the backward pass keeps.) */
#define ENTMAX_ATTN_SAVED_SLOTS 32
size_t entmax_attn_saved_bytes(const entmax_attn_params* params);
int entmax_attn_save_supports(const entmax_attn_params* params, const void* fwd_workspace, void* saved,
                              size_t saved_bytes, void* cuda_stream);

int entmax_attn_fwd_ex(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                       const float* beta, const float* gamma, const float* delta, const entmax_attn_extras* extras,
                       void* o, float* tau, void* workspace, size_t workspace_bytes, int32_t* device_status,
                       void* cuda_stream);
int entmax_attn_bwd_ex(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                       const float* beta, const float* gamma, const float* delta, const entmax_attn_extras* extras,
                       const float* tau, const void* d_o, void* dq, void* dk, void* dv, void* workspace,
                       size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

/* Where a finished forward call leaves the support of every row inside its workspace (App. A: the
 * support of row i is {j : (alpha-1) s_ij > tau_i}).  Byte offsets from the workspace base:
 *   row_count  int32 [batch*heads*seq]: support size of the row, or -2 when the row was computed by the
 *              dense path and its list is not kept (a row goes there when one of its two candidate
 *              half-lists could not be kept at `keep_limit` entries at some point of the sweep)
 *   dense_count int32 [batch*heads*seq][2]: for a row with row_count == -2, the number of keys with p > 0
 *              counted by each of the two threads that formed the row's probabilities; their sum is the
 *              support size (other rows: unspecified)
 *   entries    {float y; int32 j;} [batch*heads*seq][capacity]: the first row_count slots hold the
 *              support, y = (alpha-1) s_ij as the kernel computed it (fp32), in no particular order
 *   scale      float32 [heads*seq]: c_i
 * No paper counterpart (debugging / verification aid). */
typedef struct {
  size_t row_count_offset;
  size_t entries_offset;
  size_t scale_offset;
  size_t dense_count_offset;
  int32_t capacity;
  int32_t keep_limit; /* see row_count                                                                        */
} entmax_attn_ws_layout;
int entmax_attn_workspace_layout(const entmax_attn_params* params, entmax_attn_ws_layout* out);

/* Decode-shape forward (inference with a key/value cache): q_len new query rows per sequence against
 * that sequence's cached keys and values, sequences of different lengths in one batch.  The paper
 * evaluates its models at contexts far beyond the training length (Sec. 4, App. G: up to 65K tokens);
 * generating there means exactly this shape.  Query t of sequence b sits at position
 * pos = kv_len[b] - q_len + t, sees the keys j <= pos (causal among the new rows), and is row pos of the
 * full causal problem: Eq. 1 on s_j = c (sm_scale <q,k_j> - m_h (pos - j)), c from Eq. "asentmax" with
 * n = pos + 1 (c = delta_h for n = 1), the ALiBi term only if slopes are given.
 *   q            in,  device bf16 [batch, heads, q_len, head_dim] contiguous; 1 <= q_len <= ENTMAX_ATTN_DECODE_MAX_Q
 *   k, v         in,  device bf16 [batch, heads, kv_capacity, head_dim] with element strides
 *                kv_stride_b/h/n (all 0 = contiguous; multiples of 8; head_dim innermost), the same for both
 *   kv_len       in,  device int32 [batch], q_len <= kv_len[b] <= kv_capacity (the new rows' keys included);
 *                NULL = every sequence has kv_capacity keys.  A value outside the range sets
 *                ENTMAX_ATTN_FLAG_BAD_LENGTH in device_status and is clamped into it.
 *   beta, gamma, delta   in, device float32 [heads]; all three or none
 *   alibi_slopes in,  device float32 [heads] or NULL
 *   o            out, device bf16 [batch, heads, q_len, head_dim] contiguous
 *   tau          out, device float32 [batch, heads, q_len]
 *   support_size out, device int32 [batch, heads, q_len] or NULL: number of keys with p > 0
 *   workspace    device scratch, 256-byte aligned, >= entmax_attn_decode_workspace_bytes(params)
 *                (one fp32 score per query row and cached key, chunk maxima)
 * K is read once (the HBM traffic that bounds this shape), V only on the support.  Results are
 * bitwise reproducible.  device_status word ENTMAX_ATTN_STATUS_DENSE_ROWS counts query rows whose
 * candidate set did not fit on chip (they are solved on the score row in the workspace instead).
 * Errors as for entmax_attn_fwd; bf16 only. */
#define ENTMAX_ATTN_DECODE_MAX_Q 8
typedef struct {
  int32_t batch, heads, q_len, kv_capacity, head_dim; /* head_dim in {64, 128}                              */
  float alpha;                                         /* 1 < alpha <= 64                                    */
  float sm_scale;                                      /* 0 means 1/sqrt(head_dim)                           */
  int64_t kv_stride_b, kv_stride_h, kv_stride_n;       /* elements; all 0 = contiguous                       */
} entmax_attn_decode_params;
size_t entmax_attn_decode_workspace_bytes(const entmax_attn_decode_params* params);
int entmax_attn_decode_fwd(const entmax_attn_decode_params* params, const void* q, const void* k, const void* v,
                           const int32_t* kv_len, const float* beta, const float* gamma, const float* delta,
                           const float* alibi_slopes, void* o, float* tau, int32_t* support_size, void* workspace,
                           size_t workspace_bytes, int32_t* device_status, void* cuda_stream);

/* Forward pass for callers that cannot provide a workspace.  (The paper has no counterpart: it does
 * not discuss memory management.)
 *
 * Who needs it: code that may not, or cannot, allocate device memory at the point of the call -- a
 * plugin that is handed tensors but no allocator, a start-up or recovery path that runs before the
 * framework's memory pool exists, a region in which calling the allocator is forbidden.  Such callers
 * cannot pass the `workspace` that entmax_attn_fwd wants, so this entry point uses a fixed scratch
 * array that is part of the library image instead.  It calls no cudaMalloc / cudaFree and no
 * allocating library routine; every GPU on which the library is loaded holds
 * ENTMAX_ATTN_STATIC_SCRATCH_BYTES of device memory for it until the process exits.
 *
 * Same results as entmax_attn_fwd (O and tau; arguments as there, minus the workspace), computed by
 * the dense-row kernels: every visible key of every row is visited with fp32 arithmetic, for bf16 and
 * fp32 problems alike, so it is meant for small and medium problems, not for the long-context ones.
 *
 * Size limit: round_up(heads*seq, 32) + 64 * round_up(seq, 32) floats must fit the scratch
 * (e.g. 16 heads up to seq 26208).  Larger problems return ENTMAX_ATTN_ETOOLARGE, nothing enqueued; the size
 * is checked before the pointers are.
 *
 * Set-up: the first call on each device looks up the device address of the scratch array
 * (cudaGetSymbolAddress) with that device current; make that first call outside any stream capture.
 *
 * Sharing: all calls on a device use the same array, which keeps whatever the previous call left in it.
 * Nothing in it has to be cleared between calls (each call overwrites what it later reads), but two
 * calls that overlap on the GPU -- different streams, or different host threads without ordering --
 * race on it and produce garbage.  Calls on one stream are safe. */
#define ENTMAX_ATTN_STATIC_SCRATCH_BYTES (8u << 20)
int entmax_attn_fwd_static(const entmax_attn_params* params, const void* q, const void* k, const void* v,
                           const float* beta, const float* gamma, const float* delta, void* o, float* tau,
                           int32_t* device_status, void* cuda_stream);

/* The score-tile engine on its own (Sec. 2.1 logits before any scale): writes the raw tensor-core
 * accumulators <q_i, k_j> (bf16 inputs, fp32 accumulation) of one (batch, head) pair,
 * bh = b*heads + h, into s_out, a device float32 [seq, seq] row-major matrix, for all i and all j the
 * mask keeps; other entries are left untouched.  bf16 params only; workspace as for the forward pass.
 * Meant for verification on small seq. */
int entmax_attn_scores_debug(const entmax_attn_params* params, const void* q, const void* k,
                             int32_t bh, float* s_out, void* workspace, size_t workspace_bytes,
                             int32_t* device_status, void* cuda_stream);

/* Timing hook for benchmarks: after this call, every entmax_attn_fwd (which = 0) or entmax_attn_bwd
 * (which = 1) made by the calling thread records `start_event` immediately before and `stop_event`
 * immediately after its score-sweep kernel (bf16 problems), on that call's stream.  Both are
 * cudaEvent_t passed as void*; pass NULL for both to switch the hook off.  The events stay owned by
 * the caller.  No paper counterpart. */
int entmax_attn_profile_events(int which, void* start_event, void* stop_event);

/* Self-test of the bounded on-chip waits (no paper counterpart).  Every mbarrier wait in the tensor-core kernels gives
 * up after a time limit and makes its kernel return with ENTMAX_ATTN_FLAG_WAIT_EXPIRED in the status flags instead of
 * hanging the GPU.  This call runs one small CTA that waits, through that same code, on a barrier nothing arrives on,
 * with `limit_ns` (1 .. 100,000,000) as its limit.  On return of the kernel device_status[ENTMAX_ATTN_STATUS_FLAGS]
 * has ENTMAX_ATTN_FLAG_WAIT_EXPIRED set and device_status[1] holds the microseconds the wait lasted.
 * device_status is required here. */
int entmax_attn_selftest_wait_expiry(uint64_t limit_ns, int32_t* device_status, void* cuda_stream);

/* Text for a status code (static storage). */
const char* entmax_attn_strerror(int code);

/* The cudaError_t of the last failing CUDA call made by this library on the calling thread (0 if none). */
int entmax_attn_last_cuda_error(void);

/* Library version, major*10000 + minor*100 + patch. */
int entmax_attn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ENTMAX_ATTN_H_ */
