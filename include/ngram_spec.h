/*
 * ngram_spec.h -- C ABI of the batched N-gram speculation step for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel part of learning-free batched speculative
 * decoding ("The N-Grammys", arXiv 2411.03786):
 *
 *   draft_context_ngrams      context N-gram drafts + mixed allocation   (Sections 4.2, 4.3)
 *   build_model_ngram_tables  model bigram table and its w-token extension (Section 4.1)
 *   verify_lmhead_argmax      LM-head part of the batched verification call (Sections 3, 4.1)
 *   accept_and_commit         greedy acceptance, best row, history update  (Sections 1, 5, App. D)
 *
 * Conventions
 *   - Every function returns 0 (SPEC_OK) or a negative SPEC_ERR_* code; nothing throws or aborts.
 *     After an error spec_last_error() gives a one-line reason.
 *   - Pointers named d_* are DEVICE pointers owned by the caller, 16-byte aligned, and must stay
 *     valid until the stream work that uses them has finished.  Other pointers are host pointers.
 *     (Any device-accessible address works: small outputs such as d_acc_len / d_committed may live in
 *     mapped pinned host memory, which saves the caller a device-to-host copy per step.)
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All calls are
 *     asynchronous with respect to the host except spec_init, spec_destroy and spec_get_status.
 *   - Tokens are int32 in [0, V).  A history matrix is hist[S, cap] (row stride cap, cap % 4 == 0)
 *     with len[S] valid tokens per row.
 *   - Symbols: S sequences, B draft rows per sequence, w drafted tokens per row, q = number of
 *     trailing context tokens matched (an "N-gram" has q = N-1), V vocabulary size, d hidden
 *     size, k_tab = entries kept per row of the model bigram table, M = S*B*(w+1) verify rows.
 *   - Limits: 1 <= B <= 64, 1 <= w <= 16, 1 <= q <= 4, n_q <= 4, 1 <= topk <= B, 1 <= k_tab <= 32,
 *     d % 8 == 0, M <= SPEC_MAX_VERIFY_ROWS, history length < 2^28.
 *   - Data errors found on the device (token out of range, history overflow, a bounded wait that
 *     expired) never trap: they set bits in a status word that spec_get_status returns.
 *   - The step's kernels are launched with programmatic dependent launch: a kernel of this library
 *     may be scheduled while the previous kernel of the stream is still running, but it waits for
 *     that kernel to finish before it reads anything but the model weights.  Stream order is kept
 *     for every buffer; other work enqueued before or after behaves as with ordinary launches.
 *   - The GPU must be compute capability 10.0 (sm_100a).  There is no CPU fallback: every entry
 *     point fails with SPEC_ERR_CUDA when no such device is usable.
 *   - Host threads: a context is used by one host thread at a time (it caches tensor maps and keeps
 *     its error text); different contexts may be driven from different threads at the same time --
 *     the library's process-wide caches are locked, and spec_last_error(NULL) is per thread.  The
 *     library reads no environment variables.
 */
#ifndef NGRAM_SPEC_H_
#define NGRAM_SPEC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spec_ctx spec_ctx;

enum {
    SPEC_OK = 0,
    SPEC_ERR_ARG = -1,         /* null / misaligned pointer, size out of the documented limits */
    SPEC_ERR_UNSUPPORTED = -2, /* valid request the library does not implement */
    SPEC_ERR_CUDA = -3,        /* a CUDA runtime / driver call failed, or no sm_100 device */
    SPEC_ERR_NOT_BUILT = -4    /* model fill requested before build_model_ngram_tables */
};

/* bits of the device status word */
enum {
    SPEC_STATUS_TOKEN_RANGE = 1, /* a draft row (context or model) held a token outside [0, V): the row was dropped */
    SPEC_STATUS_CAPACITY = 2,    /* len > cap, or a commit did not fit: that sequence was skipped */
    SPEC_STATUS_TIMEOUT = 4,     /* a bounded device-side wait expired; results of that call are invalid */
    SPEC_STATUS_GROUPS = 8,      /* more distinct continuations than the drafter can group exactly */
    SPEC_STATUS_INDEX = 16       /* a context index could not take a window: that sequence is drafted by scanning until the index is rebuilt */
};

enum { SPEC_F32 = 0, SPEC_BF16 = 1 };
enum { SPEC_FLAG_DEDUP = 1, SPEC_FLAG_MODEL_FILL = 2, SPEC_FLAG_KEY_NEXT_TOKEN = 4, SPEC_FLAG_PARTIAL_TAIL = 8 };
/* OR into the draft flags to reserve n (0..255) of the B draft rows for the model strategy */
#define SPEC_FLAG_RESERVE(n) (((n) & 0xFF) << 8)
enum { SPEC_MAX_VERIFY_ROWS = 65536 };
enum { SPEC_NOALLOC_MAX_ROWS = 4096 }; /* row limit of verify_lmhead_argmax_noalloc */

/*
 * Create a context for one model head on one device.
 *   d_embed    [V, d] input embedding matrix (the paper's V, Section 4.1), row-major.
 *   d_unembed  [V, d] output embedding = lm_head weight (the paper's U^T), row-major.
 *   dtype      SPEC_BF16: both matrices are bfloat16 and are BORROWED (not copied; keep them alive).
 *              SPEC_F32 : both are float32; the context OWNS a bfloat16 copy rounded once,
 *                         round-to-nearest-even, which is what every contraction then reads.
 *   device     CUDA device ordinal; `stream` orders the conversion copy.
 * Allocates the context's scratch (verify merge keys, status word).  Synchronises the stream.
 */
int spec_init(spec_ctx** out, const void* d_embed, const void* d_unembed, int dtype, int V, int d, int device,
              void* stream);

/* Frees everything the context owns.  The caller must have finished all stream work first. */
int spec_destroy(spec_ctx* ctx);

/* Synchronises `stream`, returns the accumulated SPEC_STATUS_* bits in *status_bits and clears them. */
int spec_get_status(spec_ctx* ctx, int* status_bits, void* stream);

/* One-line description of the last error returned for this context (ctx may be NULL: global). */
const char* spec_last_error(spec_ctx* ctx);

/*
 * Model bigram table (Section 4.1 "Bigram", "Batched drafts", "Extensions").
 * For every token x: the k_tab largest entries of row x of Z = A * unembed^T, value descending,
 * equal values by ascending token id.  A = d_rows if given ([V, d] bfloat16: the model's final
 * hidden state after each single-token context), else the context's embedding matrix.
 * bf16 x bf16 products accumulate in fp32 on the tensor cores; Z is never written to memory.
 *   d_tab_idx  [V, k_tab] int32 out (required).  The context remembers this pointer (and d_ext)
 *              for draft_context_ngrams; keep it alive.
 *   d_tab_val  [V, k_tab] float32 out or NULL.
 *   d_ext      [V, k_tab, w_ext] int32 out or NULL: ext[x][r][0] = T[x][r], ext[x][r][j+1] =
 *              T[ext[x][r][j]][0] (rank-r first token, then top-1 chaining).  w_ext = 0 => none.
 * Allocates (and keeps) scratch for partial top-k lists on first use; asynchronous afterwards.
 */
int build_model_ngram_tables(spec_ctx* ctx, const void* d_rows, int k_tab, int w_ext, int32_t* d_tab_idx,
                             float* d_tab_val, int32_t* d_ext, void* stream);

/*
 * The same table built in slices, for several GPUs (rows of the table are independent: Section 4.1
 * computes p_M(.|x) one token x at a time).  Writes rows [row_begin, row_begin + row_count) of d_tab_idx
 * (and d_tab_val), which are the WHOLE [V, k_tab] arrays; d_rows, if given, is the whole [V, d] matrix.
 * Each rank builds its slice, the slices are exchanged (an all-gather of row_count * k_tab int32 per
 * rank), and spec_extend_model_table then derives the w-token extension from the complete table and
 * adopts both for draft_context_ngrams.  Nothing is adopted by build_model_ngram_table_rows itself.
 */
int build_model_ngram_table_rows(spec_ctx* ctx, const void* d_rows, int row_begin, int row_count, int k_tab,
                                 int32_t* d_tab_idx, float* d_tab_val, void* stream);
int spec_extend_model_table(spec_ctx* ctx, const int32_t* d_tab_idx, int k_tab, int w_ext, int32_t* d_ext, void* stream);

/*
 * Model unigram (Section 4.1 "Unigram").  d(x) = || u_x - ubar ||_V: u_x is row x of the unembedding,
 * ubar the mean row, and the norm is induced by <a, b>_V = sum_y (a . v_y)(b . v_y) over the rows v_y
 * of the embedding.  p(x) is proportional to exp(-d(x)), so the top-k unigram tokens are the k with the
 * smallest d.  The centred rows are rounded once to bfloat16 and contracted with the embedding on the
 * tensor cores (fp32 accumulation); the [V, V] products are squared and summed in the epilogue.
 *   d_dist2    [V] float32 out: d(x)^2.
 *   d_uni_idx  [k_uni] int32 out: tokens by ascending d, equal values by ascending id (k_uni = 0: skip).
 * Allocates (and keeps) a [V, d] bfloat16 scratch for the centred rows on first use.
 */
int build_model_unigram(spec_ctx* ctx, int k_uni, int32_t* d_uni_idx, float* d_dist2, void* stream);

/* Adopt a table built earlier (e.g. loaded from disk) instead of building it. */
int spec_set_model_table(spec_ctx* ctx, const int32_t* d_tab_idx, int k_tab, const int32_t* d_ext, int w_ext);

/*
 * Drafting (Sections 4.2 and 4.3).  Per sequence and per q in qs (caller's priority order): every
 * earlier full window of q+w tokens whose first q tokens equal the last q tokens of the history
 * is a match; matches are grouped by their w-token continuation; groups are ranked by count
 * descending, ties by the later occurrence; the first topk continuations become draft rows.
 * Rows are taken in qs order; with SPEC_FLAG_DEDUP a row equal to an earlier row is skipped; with
 * SPEC_FLAG_MODEL_FILL the remaining rows are the extended model bigram of the last token in rank
 * order.  Histories shorter than q+w give no rows for that q.  SPEC_FLAG_RESERVE(n) caps the context
 * rows at B - n so that n rows are left to the model strategy (the allocation between strategies is
 * an open knob in the paper, Section 5.2); a model row is then compared with the rows taken only.
 * SPEC_FLAG_KEY_NEXT_TOKEN groups the matches by their next token only (counting "the tokens that
 * follow each occurrence"); the row of a group is then the w tokens after its latest occurrence.
 * SPEC_FLAG_PARTIAL_TAIL also counts the occurrences that have fewer than w (but at least one) tokens
 * after them - the most recent repeats, which full windows cannot see; such a continuation is read as if
 * the history went on repeating the tokens it has (token t beyond the end = token t mod d of the d that
 * exist).  Histories then need q + 1 tokens to give rows for q.  Not available from the context index.
 *   qs         host array of n_q query lengths (n_q = 0: model rows only).
 *   d_drafts   [S, B, w] out, unused rows = -1.      d_ndrafts [S] out.
 *   d_src      [S, B] out or NULL: q of the producing strategy, 0 = model, -1 = unused.
 *   d_counts   [S, B] out or NULL: occurrence count of a context row, 0 otherwise.
 */
int draft_context_ngrams(spec_ctx* ctx, const int32_t* d_hist, const int32_t* d_len, int S, int cap,
                         const int* qs, int n_q, int topk, int B, int w, int flags, int32_t* d_drafts,
                         int32_t* d_ndrafts, int32_t* d_src, int32_t* d_counts, void* stream);

/*
 * Incremental context index (Section 4.2 defines the context N-gram as a search of the whole context at
 * every step; Section 3 wants drafting to cost next to nothing).  The index keeps, per sequence and query
 * length, what that search would find - every group (q-gram, w-token continuation) with its count and
 * latest occurrence - in a hash table in caller-owned device memory.  accept_and_commit_indexed adds the
 * windows that a step's committed tokens completed; draft_context_ngrams_indexed looks the current q-grams
 * up instead of reading the history.  The drafts are those of draft_context_ngrams, bit for bit: whenever
 * the index cannot answer for a sequence (its length is not the one the index was last updated to, a table
 * ran out of probes [SPEC_STATUS_INDEX], or the lookup met more than 2048 groups) that sequence is drafted by
 * scanning inside the same call.
 *   spec_context_index_bytes   size of the index for S sequences of capacity cap and n_q query lengths
 *                              (1.5 to 3 16-byte slots per token of capacity and query length).
 *   spec_context_index_build   builds the index of the current histories (one-off; also the way to repair
 *                              an index that fell out of step) and registers it with the context.  qs / n_q:
 *                              the query lengths to index; w: draft width; flags: SPEC_FLAG_KEY_NEXT_TOKEN or 0.
 *   draft_context_ngrams_indexed  as draft_context_ngrams; d_index must be the registered index, w and the
 *                              key flag those it was built with, every q one of its query lengths.
 *   accept_and_commit_indexed  as accept_and_commit, followed by the index update.  Commits made by any
 *                              other call leave the index out of step (detected by the length).
 * The index assumes that the tokens already in a history never change.
 */
size_t spec_context_index_bytes(int S, int cap, int n_q);
int spec_context_index_build(spec_ctx* ctx, void* d_index, const int32_t* d_hist, const int32_t* d_len, int S, int cap,
                             const int* qs, int n_q, int w, int flags, void* stream);
int draft_context_ngrams_indexed(spec_ctx* ctx, const void* d_index, const int32_t* d_hist, const int32_t* d_len, int S, int cap,
                                 const int* qs, int n_q, int topk, int B, int w, int flags, int32_t* d_drafts,
                                 int32_t* d_ndrafts, int32_t* d_src, int32_t* d_counts, void* stream);
int accept_and_commit_indexed(spec_ctx* ctx, void* d_index, const int32_t* d_drafts, const int32_t* d_ndrafts,
                              const int32_t* d_argmax, int S, int B, int w, int32_t* d_hist, int32_t* d_len, int cap,
                              int32_t* d_acc_len, int32_t* d_best_row, int32_t* d_committed, void* stream);

/*
 * Verification head (Section 3: the model call on a (k, w+1) block; here its LM-head part).
 * d_argmax[m] = argmax_y <hidden[m, :], unembed[y, :]>, lowest y on exact ties; the [M, V] logits
 * are never written.  Row m = (s*B + b)*(w+1) + j holds the hidden state at column j of draft row
 * b of sequence s (column 0 = the last context token).
 *   d_hidden   [M, d] bfloat16.      d_max  [M] float32 out or NULL (the winning logit).
 * Uses the context's merge keys as scratch: calls on one context must not overlap on the GPU.
 * If a bounded device-side wait expires (SPEC_STATUS_TIMEOUT), every row of d_argmax is -1.
 */
int verify_lmhead_argmax(spec_ctx* ctx, const void* d_hidden, int M, int32_t* d_argmax, float* d_max,
                         void* stream);

/*
 * Greedy acceptance and commit (Section 1: accept what the model would have predicted;
 * Appendix D: keep the row with the longest accepted speculation; Section 5: tokens per call).
 * a_b = longest prefix of draft row b with drafts[b][j] == argmax[b][j]; best row = largest a_b,
 * lowest b on ties (row 0, a = 0 when the sequence has no drafts).  Appends the a accepted tokens
 * and the bonus token argmax[b*][a] to the history and adds a+1 to len.  A sequence whose history
 * cannot take a+1 more tokens is left untouched, reports acc_len = best_row = -1 and sets
 * SPEC_STATUS_CAPACITY.
 *   d_argmax    [S, B, w+1] from verify_lmhead_argmax.
 *   d_acc_len   [S] out.   d_best_row [S] out.   d_committed [S, w+1] out, padded with -1.
 */
int accept_and_commit(spec_ctx* ctx, const int32_t* d_drafts, const int32_t* d_ndrafts, const int32_t* d_argmax,
                      int S, int B, int w, int32_t* d_hist, int32_t* d_len, int cap, int32_t* d_acc_len,
                      int32_t* d_best_row, int32_t* d_committed, void* stream);

/*
 * verify_lmhead_argmax followed by accept_and_commit as one call (Section 4.1 step iii plus the
 * acceptance rule above).  M = S*B*(w+1) rows of hidden states.  For up to 256 sequences the CTA
 * that merges the per-slice arg maxima also accepts and commits, so the step needs one launch
 * less; larger batches run the two kernels back to back.  Arguments as in the two calls.
 */
int verify_accept_commit(spec_ctx* ctx, const void* d_hidden, const int32_t* d_drafts, const int32_t* d_ndrafts, int S,
                         int B, int w, int32_t* d_argmax, int32_t* d_hist, int32_t* d_len, int cap,
                         int32_t* d_acc_len, int32_t* d_best_row, int32_t* d_committed, void* stream);

/*
 * Verification with the vocabulary sharded over several GPUs (one context per shard, each holding
 * V_local rows of the unembedding that start at token id vocab_offset).  verify_lmhead_keys leaves,
 * per row, a 64-bit key that orders as a signed integer by (logit, then lower global token id); the
 * caller takes the element-wise maximum over the shards (e.g. an NCCL all-reduce with max on int64)
 * and spec_unpack_keys turns the result into token ids and logits.  The paper runs on one GPU
 * (Section 5); this is the natural split of its verification call for a head that is sharded.
 *   d_keys [M] int64 out / in.   V_total = full vocabulary size (ids are clamped to it).
 */
int verify_lmhead_keys(spec_ctx* ctx, const void* d_hidden, int M, int vocab_offset, long long* d_keys, void* stream);
int spec_unpack_keys(const long long* d_keys, int M, int V_total, int32_t* d_argmax, float* d_max, void* stream);

/*
 * Ablation counters (Section 5.2: distribution of the accepted length, rank of the accepted draft
 * among the rows, rows allocated to each strategy).  Adds one decode step's outcome to running
 * histograms: d_stats = int64 [w+1] accepted length | [B] index of the accepted row (when a > 0) |
 * [5] strategy of that row (index q, 0 = model) | [5] rows allocated per strategy.  The caller
 * zeroes d_stats once; d_src is the [S, B] strategy tag from draft_context_ngrams.
 */
int spec_accumulate_stats(spec_ctx* ctx, const int32_t* d_acc_len, const int32_t* d_best_row, const int32_t* d_src, int S,
                          int B, int w, long long* d_stats, void* stream);

/*
 * 8-bit verification head.  (The paper computes in bf16 and only remarks, in its conclusion, that the
 * method composes with quantisation; this is that combination for the memory-bound regime of
 * Section 3, where the step time is the time to stream the head once: one-byte weights halve it.)
 *
 * Format: OCP FP8 E4M3 (1-4-3 bits, bias 7, no infinities, largest finite value 448), one fp32 scale
 * per row.  Quantisation of a row x (fp32 arithmetic, round to nearest even): amax = max |x|,
 * scale = amax / 448 (1 for an all-zero row), code = E4M3 nearest to x / scale (ties to the even
 * code), a zero result stored as +0.  Logit = hscale[m] * wscale[y] * sum_t hq[m][t] * wq[y][t]; the
 * products are exact and accumulate in fp32 on the tensor cores (tcgen05 kind::f8f6f4).
 *
 *   spec_quantize_rows_fp8   d_rows [n_rows, d] bfloat16 -> d_codes [n_rows, d] uint8, d_scale [n_rows].
 *   spec_quantize_head_fp8   quantises the context's unembedding into caller-owned d_wq [V, d] and
 *                            d_wscale [V] and adopts them (borrowed: keep them alive).
 *   spec_set_head_fp8        adopts a head quantised earlier.
 *   verify_lmhead_argmax_fp8 quantises d_hidden [M, d] bfloat16 into the caller's scratch d_hq [M, d],
 *                            d_hscale [M], then d_argmax[m] = argmax_y of the logit above (lowest y on
 *                            exact ties), d_max[m] (or NULL) = that logit.  Two kernels; allocates nothing.
 *                            d_hidden = NULL: d_hq / d_hscale already hold the quantised hidden states
 *                            (a model whose last layer emits them in this format); one kernel.
 * Needs d % 16 == 0 (SPEC_ERR_UNSUPPORTED otherwise); SPEC_ERR_NOT_BUILT before a head is set.
 * The result can differ from verify_lmhead_argmax wherever the two largest bf16 logits are closer
 * than the quantisation error; acceptance stays lossless with respect to the quantised model only.
 */
int spec_quantize_rows_fp8(spec_ctx* ctx, const void* d_rows, int n_rows, uint8_t* d_codes, float* d_scale, void* stream);
int spec_quantize_head_fp8(spec_ctx* ctx, uint8_t* d_wq, float* d_wscale, void* stream);
int spec_set_head_fp8(spec_ctx* ctx, const uint8_t* d_wq, const float* d_wscale);
int verify_lmhead_argmax_fp8(spec_ctx* ctx, const void* d_hidden, int M, uint8_t* d_hq, float* d_hscale,
                             int32_t* d_argmax, float* d_max, void* stream);

/*
 * Test aid: the same tensor-core main loop as the two head calls with a plain store epilogue.
 * d_logits[i, y] = <rows[i, :], unembed[y, :]> for i < m, as float32 [m, V].
 */
int spec_debug_logits(spec_ctx* ctx, const void* d_rows, int m, float* d_logits, void* stream);

/*
 * Verification head for callers that must not allocate.  (The paper has no counterpart: this is
 * a packaging variant of verify_lmhead_argmax, same kernel, same result.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they verify drafts: a
 * serving engine that has already handed all device memory to its own pool, a plug-in invoked
 * where an allocation's implicit device-wide synchronisation would stall other streams, or code
 * that is simply forbidden to change the memory map at run time.  Such callers cannot create a
 * context (spec_init allocates), so this entry point takes the unembedding matrix directly and
 * keeps its cross-CTA merge scratch in a fixed array inside the library image instead.
 *
 *   d_unembed  [V, d] bfloat16 lm_head weight, borrowed.   d_hidden [M, d] bfloat16.
 *   d_argmax   [M] int32 out.   d_max [M] float32 out or NULL.   device = CUDA ordinal.
 *
 *   - M may not exceed SPEC_NOALLOC_MAX_ROWS; a larger M is rejected with SPEC_ERR_ARG.  The array
 *     (about 33 KB) is held by every GPU that loads the library, until the process exits.
 *   - It calls no cudaMalloc / cudaFree and no routine that allocates device memory; it enqueues
 *     three small memsets and one kernel on `stream`.  ("Allocates nothing" is about device memory:
 *     the first call for a new block height may add an entry to a small host-side table.)
 *   - The first call on each device looks up the array's device address and the driver's
 *     tensor-map encoder; make that first call before any stream capture begins.  The set-up is
 *     locked, so two host threads may both make "the first call".
 *   - All calls share the one array and it keeps the previous call's contents, so the call clears
 *     what it needs first.  Two calls whose GPU work overlaps (different streams, or different
 *     threads) race on it: serialise them.
 *   - If a bounded device-side wait expires inside the kernel, every row of d_argmax is -1 (and
 *     d_max is -inf): the call has no status word a caller could read, so -1 is its error signal.
 */
int verify_lmhead_argmax_noalloc(const void* d_unembed, int V, int d, const void* d_hidden, int M,
                                 int32_t* d_argmax, float* d_max, int device, void* stream);

/*
 * Test aid for the bounded device-side waits.  Every wait inside the kernels (on an mbarrier that a
 * copy or the tensor cores complete) gives up after a time limit, sets SPEC_STATUS_TIMEOUT and lets the
 * kernel return, so that a lost completion cannot hang the GPU.  This call runs a one-thread kernel that
 * waits, with that same routine and a limit of limit_ns (at most one second), on a barrier nobody arrives
 * at: afterwards spec_get_status reports SPEC_STATUS_TIMEOUT and the context is usable as before.  With
 * mark_verify_incomplete != 0 the kernel also registers itself the way a contraction CTA that gave up
 * does, so the NEXT verify_lmhead_argmax on this context reports every row as -1 (d_max = -inf, exported
 * keys = the smallest key) instead of a partial arg max; the verification after that is normal again.
 */
int spec_debug_expire_wait(spec_ctx* ctx, unsigned long long limit_ns, int mark_verify_incomplete, void* stream);

/* Number of kernels the library has launched for this context since spec_init. */
long long spec_launch_count(spec_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* NGRAM_SPEC_H_ */
