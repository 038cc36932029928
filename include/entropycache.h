/*
 * libentropycache -- C ABI of the cached denoising step of EntropyCache
 * (training-free KV caching for diffusion language models) on NVIDIA B200 (sm_100a).
 *
 * Three operations make up the data-parallel hot path of one denoising step:
 *
 *   ec_kv_refresh    scatter the active rows' freshly projected K/V into the
 *                    full-context KV cache, in place          (Section 4.2; Appendix A, partial branch)
 *   ec_attend        refresh, then bidirectional attention in which only the
 *                    active rows are queries and every cached position is a key
 *                                                              (Appendix A: TransformerBlock(Q[M u R], K[I], V[I]))
 *   ec_entropy_gate  per-row softmax statistics of the logits (argmax,
 *                    confidence, Shannon entropy), maximum entropy over the
 *                    newly decoded rows, comparison with tau   (Eq. 1; Algorithm 1)
 *
 * and one keeps the loop's state on the device between steps:
 *
 *   ec_select_recent decode history, recent-token set R, skip_flag / dt bookkeeping and
 *                    the next partial step's row list          (Eq. 2-3; Appendix A)
 *
 * "Active rows" are the mask tokens of the current block/window plus the k most
 * recently decoded tokens (M u R); on a recompute step every row is active.
 *
 * General rules
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; the library
 *     never allocates or frees device memory and keeps no pointer after a call
 *     returns.  Descriptors (ec_attn_desc) are HOST structures, read during the call.
 *   - Every call only enqueues work on `stream` (a cudaStream_t passed as void*;
 *     NULL is the legacy default stream) and returns without synchronising.
 *   - Tensors are dense and contiguous in the layouts given below.  Every base
 *     pointer and every row (head_dim elements; a logits row) must start on a
 *     16-byte boundary.
 *   - The return value reports what the host can detect (null pointers, shapes,
 *     alignment, workspace size, launch failure).  Conditions only the device can
 *     see (a bounded wait that ran out) are written to the optional `dev_status`
 *     word; kernels never trap.
 *   - A workspace must be zero-filled once before its first use (ec_workspace_init
 *     or any memset); calls leave it ready for the next call.  Two calls that may
 *     overlap on the GPU need separate workspaces.
 */
#ifndef ENTROPYCACHE_H_
#define ENTROPYCACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EC_OK = 0,
    EC_ERR_NULL = 1,        /* a required pointer is NULL */
    EC_ERR_SHAPE = 2,       /* a size is non-positive, inconsistent or out of range */
    EC_ERR_DTYPE = 3,       /* unknown ec_dtype */
    EC_ERR_ALIGN = 4,       /* a base pointer or row is not 16-byte aligned */
    EC_ERR_WORKSPACE = 5,   /* workspace missing or smaller than *_workspace_bytes() */
    EC_ERR_UNSUPPORTED = 6, /* valid request outside what the kernels implement */
    EC_ERR_CUDA = 7,        /* a CUDA runtime call or launch failed */
    EC_ERR_TIMEOUT = 8      /* (dev_status only) a bounded device-side wait gave up */
} ec_status;

typedef enum { EC_F32 = 0, EC_BF16 = 1 } ec_dtype;

/* gate decisions (Algorithm 1: "E <= tau" reuses the cache, otherwise full recompute) */
enum { EC_SKIP = 0, EC_RECOMPUTE = 1 };

/* Geometry of one layer's attention (host structure). */
typedef struct {
    int32_t batch;       /* sequences, >= 1 */
    int32_t ctx_len;     /* L: prompt + generation positions held in the cache */
    int32_t n_q_heads;   /* H_q */
    int32_t n_kv_heads;  /* H_kv; H_q % H_kv == 0; query head h reads kv head h / (H_q/H_kv) */
    int32_t head_dim;    /* D: 64 or 128 */
    int32_t dtype;       /* ec_dtype of q, k_new, v_new, the caches and out */
    float   scale;       /* softmax scale; 0 means 1/sqrt(head_dim) */
    uint32_t flags;      /* EC_ATTN_* bits; 0 is always correct */
} ec_attn_desc;

/* (No counterpart in the paper: a scheduling permission.)  The caller states that no work still in flight on the
 * stream when ec_attend starts writes k_cache or v_cache -- typically the kernel enqueued right before the call is
 * the projection that produced q, k_new and v_new, or the attention of another layer with caches of its own.  The
 * kernels are launched with programmatic stream serialisation; with this bit they may ask for cached K/V tiles
 * before they wait for the preceding kernel to finish (q, k_new, v_new and active_idx are always read after that
 * wait).  Do not set it when the preceding work on the stream may still be writing these caches, e.g. an
 * ec_kv_refresh or ec_attend on the same caches enqueued immediately before. */
#define EC_ATTN_CACHE_SETTLED 1u

/* Layouts
 *   k_cache, v_cache  [batch, n_kv_heads, ctx_len, head_dim]
 *   k_new, v_new      [batch, n_active,  n_kv_heads, head_dim]   (post-RoPE K)
 *   q, out            [batch, n_active,  n_q_heads,  head_dim]   (post-RoPE Q)
 *   active_idx        int32 [batch, n_active]; positions in [0, ctx_len), unique
 *                     within a sequence (duplicates: the surviving row is
 *                     unspecified).  An entry outside [0, ctx_len), such as the -1
 *                     padding ec_select_recent writes, refreshes nothing; its row of
 *                     `out` is unspecified.  NULL means the identity list
 *                     0..ctx_len-1 and requires n_active == ctx_len (recompute step).
 */

/* Section 4.2 / Appendix A (partial branch): the active rows get fresh K,V, every
 * other position keeps its cached K,V.
 *     k_cache[b, h, active_idx[b,i], :] = k_new[b, i, h, :]     (same for V)
 * Bytes are copied verbatim.  n_active == 0 is a no-op.  Indices outside
 * [0, ctx_len) are skipped by the kernel (never written). */
ec_status ec_kv_refresh(const ec_attn_desc *desc, void *k_cache, void *v_cache,
                        const void *k_new, const void *v_new,
                        const int32_t *active_idx, int32_t n_active, void *stream);

/* Bytes of workspace ec_attend needs for this geometry and n_active (0 on bad arguments). */
size_t ec_attend_workspace_bytes(const ec_attn_desc *desc, int32_t n_active);

/* Appendix A, partial branch (and its full branch when n_active == ctx_len):
 *   1. if k_new/v_new are given: refresh as ec_kv_refresh does;
 *   2. out[b,i,hq,:] = sum_j softmax_j( scale * <q[b,i,hq,:], k_cache[b,hq/g,j,:]> ) * v_cache[b,hq/g,j,:]
 *      over ALL j in [0, ctx_len), no mask (bidirectional attention), reading the
 *      refreshed cache.  bf16 inputs: fp32 accumulation, bf16 output; fp32 inputs:
 *      fp32 throughout.
 * k_new and v_new may both be NULL to attend without refreshing.  workspace: at
 * least ec_attend_workspace_bytes() bytes, 16-byte aligned, zero-filled before
 * first use.  dev_status (nullable, device int32): set to an ec_status by the
 * kernels if a bounded wait ran out; untouched otherwise.  When *dev_status is non-zero after the call has
 * completed, `out` and the refreshed cache rows of that call are unspecified: always pass dev_status where a
 * wrong row must not go unnoticed (with NULL a timed-out step returns whatever it had computed). */
ec_status ec_attend(const ec_attn_desc *desc, const void *q, const void *k_new, const void *v_new,
                    void *k_cache, void *v_cache, const int32_t *active_idx, int32_t n_active,
                    void *out, void *workspace, size_t workspace_bytes,
                    int32_t *dev_status, void *stream);

/* (No counterpart in the paper: a host-only query for tests and reports.)
 * Describes the launch ec_attend would make for this geometry: the kernel's name with its template instantiation,
 * then "grid=(x,y) cluster=c ..." for the tensor-core kernels, e.g. "attend_skip_keys_kernel<48> grid=(4,32)
 * cluster=4 ring_slots=6 smem=...".  with_fresh_kv: k_new/v_new would be given; with_index_list: active_idx would be
 * non-NULL.  Touches no device memory and launches nothing.  Returns "" on arguments ec_attend would reject.  The
 * string lives in a thread-local buffer that the next call on the same thread overwrites. */
const char *ec_attend_kernel_name(const ec_attn_desc *desc, int32_t n_active, int32_t with_fresh_kv,
                                  int32_t with_index_list);

/* Bytes of workspace ec_entropy_gate needs (0 on bad arguments). */
size_t ec_entropy_gate_workspace_bytes(int32_t n_rows, int32_t vocab);

/* Eq. 1 and Algorithm 1.  For every logits row r (one pass over the row):
 *     argmax_out[r]  = smallest j maximising logits[r, j]
 *     conf_out[r]    = softmax(logits[r, :])[argmax]
 *     entropy_out[r] = - sum_j p_j ln p_j          (nats; p = softmax of the row)
 * and for every sequence b (rows b*rows_per_seq .. (b+1)*rows_per_seq - 1):
 *     max_entropy_out[b] = max over rows with decoded_flags[r] != 0 of entropy (-inf if none)
 *     decision_out[b]    = EC_RECOMPUTE if max_entropy_out[b] > tau else EC_SKIP
 * logits: [n_rows, row_stride_elems] of `dtype`, only the first `vocab` columns of
 * a row are read; -inf entries are allowed (probability 0), +inf/NaN are not.
 * argmax_out / conf_out / entropy_out may each be NULL.  n_rows must be a
 * multiple of rows_per_seq.  Arithmetic is fp32.  workspace as for ec_attend.
 * The kernel's waits on its own staged copies are bounded (one second); should one ever give up, the sequences
 * it touched get decision_out[b] = -1 (neither EC_SKIP nor EC_RECOMPUTE) and unspecified per-row outputs, and the
 * workspace stays reusable.  The same holds for the other gate entry points below. */
ec_status ec_entropy_gate(const void *logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                          int64_t row_stride_elems, int32_t rows_per_seq,
                          const uint8_t *decoded_flags, float tau,
                          int32_t *argmax_out, float *conf_out, float *entropy_out,
                          float *max_entropy_out, int32_t *decision_out,
                          void *workspace, size_t workspace_bytes, void *stream);

/* ec_entropy_gate with the other two candidate metrics of Section 5.3 ("Choice of Thresholding Variable") as
 * extra per-sequence outputs, over the same set D of decoded rows:
 *     entropy_sum_out[b] = sum over D of entropy   (0 if D is empty)
 *     max_conf_out[b]    = max over D of conf      (-inf if D is empty)
 * decision_out still applies Eq. 1's rule to the maximum entropy; thresholding the other two is the caller's.
 * Either extra pointer may be NULL.  rows_per_seq is limited to EC_GATE_DECODE_MAX_ROWS_PER_SEQ when one of them
 * is given (EC_ERR_UNSUPPORTED beyond).  Everything else as for ec_entropy_gate. */
ec_status ec_entropy_gate_metrics(const void *logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                                  int64_t row_stride_elems, int32_t rows_per_seq,
                                  const uint8_t *decoded_flags, float tau,
                                  int32_t *argmax_out, float *conf_out, float *entropy_out,
                                  float *max_entropy_out, int32_t *decision_out,
                                  float *entropy_sum_out, float *max_conf_out,
                                  void *workspace, size_t workspace_bytes, void *stream);

/* Largest rows_per_seq ec_entropy_gate_decode accepts. */
#define EC_GATE_DECODE_MAX_ROWS_PER_SEQ 64

/* The gate with confidence-based parallel decoding in front of it (Section 2.1 of the paper; its experiments use
 * the threshold 0.9): the set D of newly decoded rows, which ec_entropy_gate takes as input, is formed inside the
 * launch from the rows' confidences.  Per sequence b, with conf and argmax as ec_entropy_gate defines them:
 *     decoded[r] = masked[r] != 0 && conf[r] > conf_threshold               (fp32 comparison)
 *     if no row of the sequence qualifies and some row is masked: decoded[r*] = 1 for the masked row r* of the
 *     highest confidence, the smallest index on ties (a step decodes at least one token while any is masked)
 *     tokens[r] = argmax[r] and masked[r] = 0 for the decoded rows (other entries untouched)
 *     decoded_flags_out[r] = decoded[r]   (the array ec_select_recent takes)
 *     max_entropy_out[b] = max entropy over the decoded rows (-inf if none); decision_out[b] as ec_entropy_gate.
 * masked: uint8 [n_rows], in/out; decoded_flags_out: uint8 [n_rows]; tokens: int32 [n_rows], in/out.
 * rows_per_seq > EC_GATE_DECODE_MAX_ROWS_PER_SEQ returns EC_ERR_UNSUPPORTED.  Everything else (logits, optional
 * row outputs, workspace, errors) as for ec_entropy_gate. */
ec_status ec_entropy_gate_decode(const void *logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                                 int64_t row_stride_elems, int32_t rows_per_seq,
                                 uint8_t *masked, float conf_threshold, float tau,
                                 uint8_t *decoded_flags_out, int32_t *tokens,
                                 int32_t *argmax_out, float *conf_out, float *entropy_out,
                                 float *max_entropy_out, int32_t *decision_out,
                                 void *workspace, size_t workspace_bytes, void *stream);

/* Largest n_rows ec_entropy_gate_static accepts. */
#define EC_GATE_STATIC_MAX_ROWS 256

/* (The paper has no counterpart to this entry point: it is a packaging variant of
 * ec_entropy_gate, not a step of the method.)
 * ec_entropy_gate for callers that cannot allocate device memory and therefore have
 * no workspace to pass: a serving process whose HBM is fully pre-partitioned, a
 * plug-in that must not touch its host runtime's allocator, a step that cannot
 * afford the device-wide synchronisation of cudaMalloc.  Same arguments, results
 * and arithmetic as ec_entropy_gate, minus the workspace: the scratch is a
 * fixed array inside the library image (about 390 KB, resident on every GPU that
 * loads the library until the process exits).  The call allocates nothing.
 *   - n_rows > EC_GATE_STATIC_MAX_ROWS returns EC_ERR_UNSUPPORTED (use
 *     ec_entropy_gate with your own workspace); other argument errors as for
 *     ec_entropy_gate.
 *   - All calls on a GPU share the one scratch array: calls that may overlap on
 *     the GPU race with each other; order them on one stream or with events.
 *   - Each call clears the scratch words that must start at zero (an asynchronous
 *     memset on `stream`), so a previous call's leftovers are harmless.
 *   - The first call on each device resolves the scratch's device address; make
 *     that first call outside any stream capture. */
ec_status ec_entropy_gate_static(const void *logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                                 int64_t row_stride_elems, int32_t rows_per_seq,
                                 const uint8_t *decoded_flags, float tau,
                                 int32_t *argmax_out, float *conf_out, float *entropy_out,
                                 float *max_entropy_out, int32_t *decision_out, void *stream);

/* Eq. 2: history value of a position that has not been decoded ("-infinity"). */
#define EC_H_NEVER INT32_MIN

/* Per-sequence state of the cached denoising loop (Algorithm 1; Appendix A), DEVICE memory,
 * one element per sequence; the caller initialises it (t = first step index, the rest 0). */
typedef struct {
    int32_t t;             /* index of the current time step */
    int32_t dt_recompute;  /* steps elapsed since the last full recomputation */
    int32_t skip_flag;     /* 1: the next step is a partial step (the gate said E <= tau) */
    int32_t n_active;      /* out: rows of the next partial step (may exceed n_cap, see below) */
} ec_step_state;

/* Eq. 2-3 and the bookkeeping of Appendix A after the decode of step t, for `batch`
 * sequences in one launch, in the paper's order:
 *   1. history[b, window_start[b] + r] = t_b  for every r < block with decoded_flags[b*block + r] != 0   (Eq. 2)
 *   2. K = the k positions of sequence b with the largest history values; tau_R = max(min over K, t_b - dt_b);
 *      R = { i : history[b, i] >= tau_R }    (Eq. 3; ties at the threshold all belong to R; with fewer than k
 *      decoded positions the minimum is "-infinity" and tau_R = t_b - dt_b; k = 0 gives the empty set)
 *   3. skip_flag_b = (decision[b] == EC_SKIP);  dt_b = skip_flag_b ? dt_b + 1 : 0;  t_b = t_b + 1
 *   4. active_idx[b, :] = the block's positions window_start[b] .. window_start[b] + block - 1, then the
 *      positions of R outside the block in ascending order, then -1 up to n_cap (ec_attend and ec_kv_refresh
 *      skip negative positions); state[b].n_active = block + |R outside the block|.  If that exceeds n_cap the
 *      list is cut at n_cap entries: the caller compares n_active with n_cap and runs a full step instead.
 * history: int32 [batch, ctx_len], EC_H_NEVER where nothing was decoded; decoded_flags: uint8 [batch * block]
 * (the array ec_entropy_gate takes); window_start, decision: int32 [batch]; active_idx: int32 [batch, n_cap].
 * All DEVICE pointers.  0 <= k <= ctx_len, block <= n_cap, and every window must lie inside [0, ctx_len]:
 * a window that does not makes the kernel leave that sequence untouched and set its n_active to -1.
 * ctx_len is limited to 16384 (EC_ERR_UNSUPPORTED beyond). */
ec_status ec_select_recent(int32_t *history, int32_t ctx_len, int32_t batch, ec_step_state *state,
                           const uint8_t *decoded_flags, const int32_t *window_start, int32_t block,
                           const int32_t *decision, int32_t k, int32_t *active_idx, int32_t n_cap,
                           void *stream);

/* ec_select_recent for sliding-window decoding (Section 2.1 of the paper; its evaluation mode, window size 32): the
 * window of a step is the first `window` still-masked positions of the sequence, so the number of mask tokens being
 * denoised stays constant while the window advances; it stops being contiguous as soon as a position inside it is
 * decoded.  Per sequence b, in one launch:
 *   1. for every r < window with decoded_flags[b*window + r] != 0: pos = active_idx[b, r] (the window the previous
 *      call wrote; before the first call the caller writes the first window there): history[b, pos] = t_b and
 *      masked[b, pos] = 0                                                                      (Eq. 2)
 *   2. K, tau_R, R exactly as ec_select_recent                                                 (Eq. 3)
 *   3. skip_flag_b, dt_b, t_b exactly as ec_select_recent                                      (Appendix A)
 *   4. active_idx[b, :] = the first `window` positions with masked[b, pos] != 0, ascending (fewer when fewer
 *      remain), then the positions of R ascending (a decoded position is never masked, so the two are disjoint),
 *      then -1 up to n_cap; state[b].n_active = their count (beyond n_cap the list is cut, as in ec_select_recent).
 * masked: uint8 [batch, ctx_len], in/out; the other arguments as for ec_select_recent.
 * Between two calls the caller changes neither `masked` nor active_idx: the size of the current window is recomputed
 * as min(window, number of masked positions of the sequence), and its rows are read back from active_idx[b, 0 : that
 * size].  Before the first call the caller writes exactly that many entries, the first masked positions in ascending
 * order.  A sequence whose current window holds an entry that is out of range or no longer masked is left untouched
 * (history, masked, state, list) except for state[b].n_active = -1. */
ec_status ec_select_recent_sliding(int32_t *history, int32_t ctx_len, int32_t batch, ec_step_state *state,
                                   uint8_t *masked, const uint8_t *decoded_flags, int32_t window,
                                   const int32_t *decision, int32_t k, int32_t *active_idx, int32_t n_cap,
                                   void *stream);

/* Zero-fills a workspace (asynchronous on `stream`). */
ec_status ec_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/* Static, human-readable name of a status code. */
const char *ec_status_string(int32_t status);

/* Library version: major * 10000 + minor * 100 + patch. */
int32_t ec_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ENTROPYCACHE_H_ */
