/*
 * libasap -- the ASAP visual-token prune step (arXiv 2603.14549, Sec. 4) for one B200 (sm_100a).
 *
 * The step runs between two decoder layers during prefill.  For every sequence of a packed
 * batch, laid out as [ prefix (system prompt) | visual span I | suffix (text) ], it
 *   1a. sums the pre-softmax alignment W = Q K^T / sqrt(d) over the visual queries to get the
 *       attention mass s_j of every visual key                                   (Sec. 4.1, Eq. 1)
 *   1b. min-max normalises s to the salience s_hat and forms the mask vector
 *       m_j = ln max(lambda_max * s_hat_j, eps)                                  (Eq. 2, Eq. 3)
 *   1c. evaluates A = Softmax(W + M_bidir) on the ranking query rows            (Eq. 3, Eq. 4)
 *   2.  averages A over heads and ranking rows into one score r_j per visual key
 *   3.  keeps the keep_k visual tokens of largest r_j (ties: lower index)        (Fig. 3)
 *   4a. sends every dropped token to the kept token of highest cosine similarity (Sec. 4.2)
 *   4b. replaces every kept token by the salience-weighted mean of itself and the tokens
 *       sent to it                                                               (Eq. 5)
 *   5.  writes the shortened sequence [ prefix | kept visual, ascending | suffix ] with its
 *       gathered position ids                                                    (Fig. 3)
 *
 * Conventions for every entry point
 *   - Pointers inside asap_inputs / asap_outputs are DEVICE pointers owned by the caller; the
 *     structs themselves and the asap_params struct live in HOST memory.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work: they never
 *     synchronise the stream, never read device memory on the host and never allocate (all
 *     scratch memory is taken by asap_init).
 *   - Every function returns an asap_status and never throws or aborts.  On ASAP_ERR_* no
 *     kernel has been launched by that call and the outputs are untouched.  The text of the
 *     last error is available from asap_last_error.
 *   - Host-side checks cover what the host can see (null pointers, 16-byte alignment of
 *     q / k / hidden / out_hidden, head_dim == 128, D == H * head_dim, 0 < keep_k <= min_vis,
 *     0 < lambda_max <= 1, eps > 0, sizes within the asap_init capacities).  The per-sample
 *     arrays live on the device; the first kernel of each call checks them (spans inside the
 *     sequence, vis_len within [min_vis, max_vis], ascending cu_seqlens, ...) and records a
 *     violation in a device status word that asap_check reads.  A kernel never traps or
 *     spins without bound; every wait in the tensor-core kernels has a limit (about a second)
 *     after which a time-out bit is set in the status word and the block leaves, once the copies
 *     and tensor-core operations it has in flight have completed.  A time-out bit is sticky: every
 *     result enqueued on the context since it was set is invalid (later tensor-core kernels see the
 *     bit and leave at once), and the context resumes normal work only after asap_check has
 *     reported and cleared the word.
 *   - bf16 tensors are row-major with the stated shapes and no padding.
 *   - A context serves one stream at a time: two calls on the same context that overlap on
 *     the GPU race on its scratch memory.
 *   - asap_prune_step may enqueue two of its kernels (attention mass, salience) on a second
 *     stream that belongs to the context, forked from and joined back into `stream` with
 *     events inside the call: everything the call enqueues is ordered after the work already
 *     in `stream`, and work enqueued in `stream` after the call is ordered after all of it.
 */
#ifndef ASAP_H
#define ASAP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct asap_ctx asap_ctx; /* opaque: scratch memory, device status word, error text */

typedef enum {
  ASAP_OK = 0,
  ASAP_ERR_INVALID = -1,     /* bad argument visible to the host */
  ASAP_ERR_ALIGN = -2,       /* a tensor pointer is not 16-byte aligned */
  ASAP_ERR_WORKSPACE = -3,   /* the problem exceeds the capacities given to asap_init */
  ASAP_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed */
  ASAP_ERR_UNSUPPORTED = -5, /* head_dim != 128, D not a multiple of 8, ... */
  ASAP_ERR_DEVICE = -6       /* asap_check: a kernel flagged bad device-side data or a timed-out wait */
} asap_status;

/* Problem description.  Sequence b owns packed rows cu_seqlens[b] .. cu_seqlens[b+1]-1.  Span
 * starts are relative to the start of their sequence. */
typedef struct {
  int32_t B;            /* sequences in the batch */
  int32_t H;            /* attention heads */
  int32_t head_dim;     /* must be 128 */
  int32_t D;            /* hidden size, == H * head_dim */
  int32_t total_tokens; /* rows of q / k / hidden / pos_ids == cu_seqlens[B] */
  int32_t min_vis;      /* host-known bounds: min_vis <= vis_len[b] <= max_vis */
  int32_t max_vis;
  int32_t max_seq;      /* bound on the length of any sequence */
  int32_t max_rank;     /* bound on rank_len[b] (on text_len[b] when rank_start is NULL) */
  const int32_t *cu_seqlens; /* [B+1] */
  const int32_t *vis_start;  /* [B] image span I */
  const int32_t *vis_len;    /* [B] */
  const int32_t *text_start; /* [B] text span, text_start >= vis_start + vis_len */
  const int32_t *text_len;   /* [B] */
  const int32_t *rank_start; /* [B] query rows whose Eq. 4 probabilities rank the visual keys; */
  const int32_t *rank_len;   /* [B] both NULL => the text span.  rank_len[b] >= 1.             */
  const void *q;             /* bf16 [total_tokens, H, head_dim], rotary embedding applied */
  const void *k;             /* bf16 [total_tokens, H, head_dim], rotary embedding applied */
  const void *hidden;        /* bf16 [total_tokens, D], hidden states after the pruning layer */
  const int32_t *pos_ids;    /* [total_tokens] */
} asap_inputs;

typedef struct {
  int32_t keep_k;       /* visual tokens kept per sequence, 0 < keep_k <= min_vis */
  float lambda_max;     /* Eq. 3 leak budget, in (0, 1] */
  float eps;            /* Eq. 2 / Eq. 3 / Eq. 5 epsilon, the paper uses 1e-6 */
  float sim_threshold;  /* Sec. 4.2 threshold t: merge only if cosine similarity > t; -INFINITY = always */
  int32_t mask_enable;  /* 0: Eq. 3 is replaced by the causal mask of Sec. 3.2 */
  int32_t merge_enable; /* 0: kept tokens are copied unmerged, assign = -1 */
  int32_t per_head_mask; /* 0: one salience and one mask for all heads, from the head-mean attention mass
                            (the reading used throughout).  1: Eq. 1-3 separately per head -- s_j^h, s_hat_j^h,
                            m_j^h -- head h's logits get head h's mask (asap_outputs::mask_log_heads), and a
                            token's Eq. 5 weight is the mean over heads of s_hat_j^h.  Needs an even H. */
} asap_params;

/* Results.  Per-sequence arrays are padded to the stated pitch; entries past vis_len[b]
 * (or past vis_len[b] - keep_k) are 0 for floats and -1 for indices.  Visual indices are
 * relative to the start of the image span. */
typedef struct {
  float *mass;       /* [B, max_vis] s_j       (Eq. 1, mean over heads)            */
  float *salience;   /* [B, max_vis] s_hat_j   (Eq. 2)                             */
  float *mask_log;   /* [B, max_vis] m_j       (Eq. 3)                             */
  float *rank_score; /* [B, max_vis] r_j       (mean over heads, ranking rows of Eq. 4) */
  int32_t *keep_idx; /* [B, keep_k]            kept visual indices, ascending      */
  int32_t *drop_idx; /* [B, max_vis - keep_k]  dropped visual indices, ascending   */
  int32_t *assign;   /* [B, max_vis - keep_k]  kept SLOT (0..keep_k-1) a dropped token merges into, or -1 */
  float *best_sim;   /* [B, max_vis - keep_k]  its cosine similarity to that slot; may be NULL */
  void *out_hidden;  /* bf16 [out_rows, D]     shortened sequences, packed         */
  int32_t *out_pos;  /* [out_rows]             position ids gathered from pos_ids  */
  int32_t *src_row;  /* [out_rows]             packed input row each output row came from */
  int32_t *out_cu_seqlens; /* [B+1]            row offsets of the shortened sequences */
  int32_t out_rows_capacity; /* rows available in out_hidden / out_pos / src_row; the step needs
                                total_tokens - sum_b vis_len[b] + B * keep_k, which is at most
                                total_tokens - B * (min_vis - keep_k) */
  float *mask_log_heads;     /* [B, H, max_vis] m_j^h; written (and required) only with per_head_mask.  In that
                                mode `mass` is the head mean of s_j^h, `salience` the head mean of s_hat_j^h and
                                `mask_log` Eq. 3 of that mean (not used by the step itself). */
} asap_outputs;

/* Creates a context on `device` and takes all scratch memory the step will ever need for
 * problems with total_tokens <= max_total_tokens, B <= max_B, H <= max_H, D <= max_D and
 * B * keep_k <= max_keep_rows (0 = max_total_tokens).  The only call that allocates.
 * Which kernel form a launch takes is decided from the problem size; four environment variables, read
 * here once per context, move those decisions for measurements (results are the same up to rounding order):
 *   ASAP_FUSE_MASS_MIN_TOKENS   B * max_vis from which Eq. 1's key side rides in the score kernel (default 50000)
 *   ASAP_SIM_PAIR_MIN_BLOCKS    blocks from which the similarity takes two row tiles per block (default: half the SMs)
 *   ASAP_SIM_PAIR_STAGES        tile stages of that form (default: what fits 192 KB)
 *   ASAP_SIM_CLUSTER            0: sliced similarity launches add their partial products through global memory
 *                               instead of a thread-block cluster's shared memory (default 1, if the device can
 *                               place such a cluster) */
asap_status asap_init(asap_ctx **ctx, int device, size_t max_total_tokens, int max_B, int max_H,
                      int max_D, size_t max_keep_rows);

/* Steps 1a-2 (Sec. 4.1, Eq. 1-4).  Writes out->mass, salience, mask_log, rank_score. */
asap_status asap_score(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                       const asap_outputs *out, void *stream);

/* Step 3 (Fig. 3: top-k retained).  Reads `rank_score` [B, max_vis]; writes out->keep_idx,
 * out->drop_idx. */
asap_status asap_select(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                        const float *rank_score, const asap_outputs *out, void *stream);

/* Steps 4a-5 (Sec. 4.2, Eq. 5; hand-off of Fig. 3).  Reads `salience`, `keep_idx`, `drop_idx`
 * (layouts as in asap_outputs); writes out->assign, best_sim (if non-NULL), out_hidden,
 * out_pos, src_row, out_cu_seqlens. */
asap_status asap_merge(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                       const float *salience, const int32_t *keep_idx, const int32_t *drop_idx,
                       const asap_outputs *out, void *stream);

/* Stage 2 in the wording of Sec. 4.2: redundancy is removed INSIDE the kept set and the freed
 * budget goes back to the pruned pool.  Given stage 1's results (`mass` s_j of Eq. 1, `salience`
 * s_hat_j of Eq. 2, the kept and pruned lists of asap_select, all device arrays laid out as in
 * asap_outputs) the call
 *   - forms the cosine similarity S of every pair of kept tokens;
 *   - visits the kept tokens by salience (descending, lower sequence index first among equals):
 *     a token whose similarity to an earlier, not absorbed token (an anchor) exceeds
 *     p->sim_threshold is absorbed by the most similar such anchor (lowest index among equals),
 *     any other token becomes an anchor; at most vis_len[b] - keep_k tokens are absorbed, so that
 *     every vacated slot can be refilled;
 *   - replaces every anchor by the salience-weighted mean of itself and its sources (Eq. 5);
 *   - refills the vacated slots with the pruned tokens of largest s_j (lower index first among
 *     equals), so that exactly keep_k visual tokens leave;
 *   - compacts hidden states and position ids as asap_merge does.
 * Outputs: out->keep_idx = the final kept list (anchors and refilled tokens, ascending);
 * out->drop_idx = the absorbed tokens, ascending, padded with -1; out->assign = the slot in
 * out->keep_idx each of them was merged into; out->best_sim (if non-NULL) = its similarity to that
 * anchor; out_hidden, out_pos, src_row, out_cu_seqlens as in asap_merge.  `n_absorbed` ([B],
 * device, may be NULL) receives the number of absorbed tokens per sequence.
 * `keep_idx` / `drop_idx` must not be the arrays `out` points to.  `scratch` is caller-owned
 * device memory of at least asap_consolidate_scratch_bytes(B, keep_k) bytes, 16-byte aligned
 * (the similarity matrix, keep_k * keep_k floats per sequence, and a bit matrix); nothing is
 * kept in it between calls.  Requires p->merge_enable and keep_k < max_vis (ASAP_ERR_INVALID
 * otherwise: asap_merge covers those cases) and keep_k <= 4096 (ASAP_ERR_UNSUPPORTED).  May be
 * recorded by a stream capture. */
size_t asap_consolidate_scratch_bytes(int32_t B, int32_t keep_k);
asap_status asap_consolidate(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                             const float *mass, const float *salience, const int32_t *keep_idx,
                             const int32_t *drop_idx, void *scratch, size_t scratch_bytes,
                             const asap_outputs *out, int32_t *n_absorbed, void *stream);

/* The layer's attention under the salience-guided bidirectional mask (Sec. 4.1, Eq. 3-4):
 *     out[i, h, :] = sum_j Softmax_j( q_i^h . k_j^h / sqrt(head_dim) + M_ij ) v_j^h
 * for every row i of every sequence, with M_ij = 0 for j <= i, M_ij = mask_log[b][j - vis_start]
 * for i < j when both i and j lie in the image span, and -infinity otherwise (other sequences of
 * the packed batch are never attended).  With p->mask_enable == 0 this is causal attention and
 * `mask_log` may be NULL; otherwise `mask_log` is the device array [B, max_vis] that asap_score
 * writes (asap_outputs::mask_log), or with p->per_head_mask the array [B, H, max_vis] of
 * asap_outputs::mask_log_heads (head h then uses its own vector).  Only B, H, head_dim, D, total_tokens, the bounds, cu_seqlens,
 * the spans, q and k of `in` are read; `p` must be a valid parameter set (as for asap_score).
 * `v` and `out` are bf16 [total_tokens, H, head_dim] device tensors, 16-byte aligned, that must
 * not overlap.  `scratch`: caller-owned device memory of at least
 * asap_attention_scratch_bytes(total_tokens, D) bytes, 16-byte aligned (the transposed values);
 * nothing is kept in it between calls.  Two launches (plus the validation kernel); may be recorded
 * by a stream capture. */
size_t asap_attention_scratch_bytes(int32_t total_tokens, int32_t D);
asap_status asap_attention(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                           const float *mask_log, const void *v, void *scratch, size_t scratch_bytes,
                           void *out, void *stream);

/* Steps 1a-5 back to back on `stream`; fills every field of `out`.  The call may be recorded by a
 * stream capture (it allocates nothing and does not synchronise; the context's side stream forks from
 * and joins back into `stream` inside the call) and the graph replayed on new contents of the same
 * buffers. */
asap_status asap_prune_step(asap_ctx *ctx, const asap_inputs *in, const asap_params *p,
                            const asap_outputs *out, void *stream);

/* KV-cache compaction (the paper presents the method as KV-cache compatible, Sec. 1, and reports
 * the key/value storage it saves, Sec. 5.5 / Table 4).  The decoder layers up to the pruning layer
 * have already cached keys and values for every token of the prompt; after the prune step only
 * the rows of the shortened sequence are needed.  For each of `n_tensors` (<= 64) row-major
 * tensors of `src_rows` rows of `row_bytes` bytes (a multiple of 16; e.g. one layer's K or V,
 * [total_tokens, kv_heads * head_dim]) this writes dst[t][r] = src[t][src_row[r]] for
 * r < *n_rows, r < rows_capacity.  `src_row` and `n_rows` are DEVICE pointers: the row map
 * written by asap_merge / asap_prune_step and the number of rows of the shortened batch
 * (out_cu_seqlens + B); `src` and `dst` are HOST arrays of device pointers, 16-byte aligned,
 * that must not overlap.  A map entry outside [0, src_rows) leaves its output row untouched.
 * Position ids of the kept rows are the gathered ones of asap_outputs::out_pos, so rotary
 * phases already baked into cached keys stay valid. */
asap_status asap_compact_kv(asap_ctx *ctx, const int32_t *src_row, const int32_t *n_rows,
                            int32_t rows_capacity, int32_t src_rows, size_t row_bytes, int32_t n_tensors,
                            const void *const *src, void *const *dst, void *stream);

/* Reads the device status word (one 4-byte copy after synchronising `stream`).  ASAP_OK, or
 * ASAP_ERR_DEVICE with the reason in asap_last_error; the word is cleared.  After a time-out bit
 * (a bounded wait ran out in a tensor-core kernel) every result enqueued on the context since
 * the bit was set is invalid, and the call also puts the kernels' hand-shake counters back to
 * zero; the context is ready for normal work when it returns. */
asap_status asap_check(asap_ctx *ctx, void *stream);

/* Text of the last error recorded on this context (empty string if none).  Valid until the
 * next call on the context.  asap_last_error(NULL) describes a failed asap_init or
 * asap_select_static; that text lives in one buffer shared by all threads of the process. */
const char *asap_last_error(const asap_ctx *ctx);

/* Step 3 once more, for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is the same top-k as asap_select, packaged differently.)
 *
 * asap_select needs a context, and asap_init takes its scratch with cudaMalloc.  Some callers
 * have no such moment: a plug-in that runs inside a host application's already-captured or
 * memory-budgeted region, a real-time loop that may not touch the allocator, a process whose
 * device memory is handed out entirely by another component.  For them this entry point keeps
 * the scratch of the selection (the per-sequence descriptors and the kept / dropped role of
 * every visual token) in a fixed array that is part of the library image: about 1 MiB on every
 * GPU that loads libasap, held until the process exits.  It calls no cudaMalloc / cudaFree and
 * no routine that allocates; the caller passes every input and output.
 *
 * Limits: B <= 64 and B * max_vis <= 262144 (ASAP_ERR_WORKSPACE beyond that, nothing launched).
 * Only the fields of `in` that asap_select reads are used: the sizes and the per-sequence
 * arrays (q, k, hidden, pos_ids may be NULL).  `rank_score`, `keep_idx`, `drop_idx` are as in
 * asap_select.  `device_status` may be NULL; otherwise it points to one caller-owned 32-bit
 * word in device memory that is cleared and then receives bit 0 if a per-sequence array entry
 * failed validation (that sequence's outputs are all -1).
 *
 * The call works on the calling thread's current device; `stream` must belong to it.  The
 * first call on a device looks the array's device address up and raises the kernel's shared
 * memory limit; make that first call outside any stream capture.  All calls on a device share
 * the one array, which keeps what the previous call left: the call clears the status word
 * itself and overwrites the rest, but two calls that overlap on the GPU (different streams,
 * different threads) race on it.  Errors are reported through asap_last_error(NULL), one text
 * buffer for the whole process: read it from the thread that made the failing call, before another
 * thread calls asap_init or this function.  With device_status == NULL a sequence that fails the
 * device-side validation is still skipped (its outputs are all -1) but nothing the caller can
 * read records that: pass a status word if the per-sequence arrays are not trusted.  The first
 * call on a device also pays for what any first CUDA call pays (context creation, loading of the
 * library's device code), which the driver does with allocations of its own. */
asap_status asap_select_static(const asap_inputs *in, const asap_params *p, const float *rank_score,
                               int32_t *keep_idx, int32_t *drop_idx, uint32_t *device_status,
                               void *stream);

/* Per-kernel device times.  Not part of the method (the paper has no counterpart): a
 * measurement aid.  asap_profile(ctx, 1) makes every later entry point drop one CUDA event on
 * its stream before each kernel and one after its last kernel (the first enabling call creates
 * the events; at most 16384 are used between two reads, later launches go untimed).
 * asap_profile(ctx, 0) stops that.  Either call clears the accumulated times. */
typedef struct {
  char name[32];     /* kernel name: "qsum", "mass_salience", "score", "select", "sim", ... */
  uint64_t launches; /* launches timed since profiling was enabled */
  double total_ms;   /* Diagnostics for the bounded waits of the tensor-core kernels (conventions above; the paper has no
 * counterpart).  The next call of an entry point on this context -- and only that call -- runs with
 * `cycles` clock cycles as the limit of every wait, instead of about a second.  With a limit of a few
 * cycles a healthy run gives up at its first wait that is not satisfied at once: the call returns
 * normally, its results are invalid, and asap_check reports ASAP_ERR_DEVICE with the kernel's
 * time-out bit.  This is how the give-up path is exercised without making anything hang.  cycles must
 * be positive. */
asap_status asap_debug_wait_limit(asap_ctx *ctx, long long cycles);

/* sum over those launches of (next event - this kernel's event) */
} asap_kernel_time;
asap_status asap_profile(asap_ctx *ctx, int enable);

/* Waits for the last recorded event, folds the events recorded since the previous read into
 * the per-kernel totals, copies up to `capacity` totals to `out` (host memory) and returns how
 * many kernels have a total.  A kernel's time runs to the start of the next kernel of the same
 * call, so it includes the launch gap behind it. */
int asap_profile_read(asap_ctx *ctx, asap_kernel_time *out, int capacity);

/* Number of kernel launches the library has enqueued through this context so far. */
uint64_t asap_launch_count(const asap_ctx *ctx);

/* Releases the context and its scratch memory.  NULL is allowed. */
void asap_free(asap_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* ASAP_H */
