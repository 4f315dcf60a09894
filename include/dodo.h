/*
 * dodo.h -- C ABI of the B200 (sm_100a) library for the inference hot path of
 * Dodo, dynamic contextual compression for decoder-only LMs (arXiv 2310.02409).
 *
 * Per transformer layer the path is
 *
 *   score    s_i = Scorer(x_i)                         Eq. 6, Eq. 15
 *   select   keep the k = ceil(n/r) best-scored tokens  Eq. 14 (+ footnote), Sec. 2.3
 *   gather   z_{1:k} = the selected tokens' K/V rows    Eq. 5, Eq. 4
 *   attend   Attn(q, [z_{1:k} ; recent local tokens])   Eq. 4, Eq. 9, Eq. 13, Eq. 16
 *
 * General conventions
 *   - Every function returns a dodo_status (0 = DODO_OK, negative = error).  Argument errors are
 *     detected on the host before anything is launched; dodo_last_error() gives the reason.
 *   - Pointers marked [device] are device memory owned by the caller (borrowed for the call, never
 *     freed or retained).  Pointers marked [host] are ordinary host arrays, read during the call
 *     and not retained; their contents are baked into kernel parameters, so the nugget count k is
 *     always known on the host and no call synchronises with the device.
 *   - Work is enqueued asynchronously on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream).
 *   - Ragged batches: sequence b owns rows [off[b], off[b+1]) of a packed array.
 *   - Tensors are row-major and dense.  Device base addresses must be 16-byte aligned and a
 *     token row (d, or H*dh elements) must be a multiple of 16 bytes.
 *   - A dodo_ctx owns a small device scratch (arrival counters).  Calls that share a ctx must be
 *     ordered on the device (same stream, or otherwise serialised); use one ctx per concurrent
 *     stream.  A ctx is not thread-safe.
 *   - Nothing on the device traps, and every wait on the device is bounded: a wait that runs out sets
 *     DODO_DEV_WAIT_TIMEOUT in the device status word and the kernel returns (dodo_device_status).
 */
#ifndef DODO_H
#define DODO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define DODO_API __attribute__((visibility("default")))
#else
#define DODO_API
#endif

typedef struct dodo_ctx dodo_ctx;

typedef enum {
    DODO_OK = 0,
    DODO_ERR_INVALID_ARG = -1, /* bad pointer, size, offset table, k > n, misalignment          */
    DODO_ERR_UNSUPPORTED = -2, /* dtype / head_dim / shape outside what the kernels are built for */
    DODO_ERR_CAPACITY = -3,    /* a cache region or the workspace is too small                   */
    DODO_ERR_CUDA = -4         /* a CUDA runtime or driver call failed                           */
} dodo_status;

typedef enum { DODO_F32 = 0, DODO_BF16 = 1 } dodo_dtype;

/* Selection flag: the last token of every sequence is always kept as a nugget (footnote to
 * Eq. 14); the other k-1 nuggets are the best-scored of the remaining tokens. */
enum { DODO_FORCE_LAST = 1u };

/* Create a context on CUDA device `device` (allocates a few hundred KB of device scratch, zeroed
 * once).  Fails with DODO_ERR_CUDA when no usable sm_100 device is present. */
DODO_API int dodo_create(dodo_ctx** out, int device);
DODO_API int dodo_destroy(dodo_ctx* ctx);

/* Human-readable reason of the last error on this context (valid until the next call). */
DODO_API const char* dodo_last_error(const dodo_ctx* ctx);

/* Re-zero the context's arrival counters and its device status word on `stream`.  Only needed after a
 * launch failed midway or a kernel reported a problem. */
DODO_API int dodo_reset(dodo_ctx* ctx, void* stream);

/* Reads the context's device status word (synchronises with the device).  0 = no kernel reported a
 * problem; otherwise a set of DODO_DEV_* bits, which stay set until dodo_reset:
 *   DODO_DEV_WAIT_TIMEOUT  a bounded wait ran out: on an asynchronous copy or a tensor-core operation
 *                          (tensor-core kernels), or on a sequence's selection flag (dodo_compress);
 *                          results of that launch are invalid, call dodo_reset before reusing the context
 *   DODO_DEV_BAD_INDEX     a gather met an index outside [0, n_b) of its sequence; that nugget's cache
 *                          row and position were left as they were, every other row is correct */
enum { DODO_DEV_WAIT_TIMEOUT = 1, DODO_DEV_BAD_INDEX = 2 };
DODO_API int dodo_device_status(dodo_ctx* ctx, int* status);

/* Performance knobs (defaults are tuned for B200; results do not depend on them beyond fp32
 * summation order).  DODO_TUNE_ATTEND_TARGET_BLOCKS: split-K aims at about this many thread blocks
 * per dodo_attend launch (default 2 x SM count); changes dodo_attend_workspace_bytes.
 * (Knob 2, a shared-memory stage count, belonged to an earlier kernel and is gone: it is refused.)
 * DODO_TUNE_DENSE_MIN_QUERIES: a call whose longest query block has at least this many tokens
 * (bf16, head size 128) runs on the tensor-core kernel (default 32); a very large value keeps
 * everything on the streaming kernel.
 * DODO_TUNE_DENSE_BALANCE: how the tensor-core kernel spreads (sequence, query tile, head) units
 * over thread blocks: 0 (default) balances key tiles over the resident blocks when the units alone
 * would leave SMs idle and the key lists are long, 1 balances whenever the workspace allows (cut
 * units meet through the workspace), 2 never does (one block per unit), 3 balances like 1 but
 * never keeps the query tiles of a head in step (each block takes its own slot range). */
enum { DODO_TUNE_ATTEND_TARGET_BLOCKS = 1, DODO_TUNE_DENSE_MIN_QUERIES = 3, DODO_TUNE_DENSE_BALANCE = 4 };
DODO_API int dodo_set_tuning(dodo_ctx* ctx, int knob, int value);

/* Number of nuggets for n context tokens at compression ratio r >= 1: k = ceil(n / r) in integer
 * arithmetic (Sec. 2.3, text before Eq. 14).  Returns -1 on n < 0 or r < 1. */
DODO_API int dodo_num_nuggets(int n, int r);

/*
 * Scorer, linear form (Eq. 6 / Eq. 15): scores[i] = sum_c X[i][c] * w[c] + bias, accumulated in
 * fp32, for every row of a ragged-packed batch.
 *   X        [device] [seq_off[B], d] in `dtype`         w  [device] [d] in `dtype`
 *   seq_off  [host]   int32[B+1], non-decreasing, seq_off[0] = 0
 *   scores   [device] float[seq_off[B]], written
 */
DODO_API int dodo_score(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
               const int32_t* seq_off, int B, float* scores, void* stream);

/*
 * Two-layer Scorer (Eq. 6 with the feed-forward network the paper describes in App. B.3, d -> dh -> 1;
 * its parameter count in Table 5 fits dh = d): s_i = w2 . act(W1 x_i + b1) + b2 for every row of X.
 * The paper does not name the activation; `act` selects it.  The first layer runs on the tensor
 * cores (bf16 inputs, fp32 accumulation); bias, activation and the product with w2 are fp32.
 *   X       [device] [seq_off[B], d] bf16, 16-byte aligned      W1 [device] [dh, d] bf16 (one row per hidden unit)
 *   b1      [device] float[dh]      w2 [device] bf16[dh]      b2 scalar
 *   scores  [device] float[seq_off[B]], written
 *   workspace [device] at least dodo_score_mlp_workspace_bytes(rows, dh) bytes, 16-byte aligned (partial scores
 *           of groups of hidden units, added in a fixed order: scores are reproducible bit for bit)
 * Supported: dtype DODO_BF16, d a multiple of 64, dh a multiple of 256; else DODO_ERR_UNSUPPORTED.
 * The scores feed dodo_select / dodo_select_threshold like those of dodo_score.
 */
enum { DODO_ACT_IDENTITY = 0, DODO_ACT_RELU = 1, DODO_ACT_GELU_TANH = 2 };
DODO_API size_t dodo_score_mlp_workspace_bytes(int rows, int dh);
DODO_API int dodo_score_mlp(dodo_ctx* ctx, const void* X, int dtype, int d, const void* W1, const float* b1,
                   const void* w2, float b2, int dh, int act, const int32_t* seq_off, int B, float* scores,
                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * dodo_score_mlp followed by dodo_select, the TopK (Eq. 14) fused into the reduction that ends the two-layer
 * Scorer: while no sequence is longer than 4096 tokens the block that adds up a sequence's last scores selects its
 * nuggets (two launches in all: the tensor-core pass, the reduction with selection); longer sequences are selected
 * by a launch of their own.  `scores` holds what dodo_score_mlp would write, idx equals dodo_select on them.
 */
DODO_API int dodo_score_mlp_select(dodo_ctx* ctx, const void* X, int dtype, int d, const void* W1, const float* b1,
                          const void* w2, float b2, int dh, int act, const int32_t* seq_off, const int32_t* nug_off,
                          int B, uint32_t flags, float* scores, int32_t* idx, void* workspace, size_t workspace_bytes,
                          void* stream);

/*
 * TopK selection (Eq. 14): for every sequence b keep the k_b = nug_off[b+1] - nug_off[b] positions
 * with the highest scores among its n_b = seq_off[b+1] - seq_off[b] tokens.  Equal scores go to the
 * lower position; -0 equals +0; NaN ranks below -inf.  The result is unique.
 *   scores   [device] float[seq_off[B]]
 *   nug_off  [host]   int32[B+1], 0 <= k_b <= n_b (k_b > n_b -> DODO_ERR_INVALID_ARG)
 *   flags    0 or DODO_FORCE_LAST
 *   idx      [device] int32[nug_off[B]], written: sequence-local positions, ascending per sequence
 */
DODO_API int dodo_select(dodo_ctx* ctx, const float* scores, const int32_t* seq_off, const int32_t* nug_off,
                int B, uint32_t flags, int32_t* idx, void* stream);

/*
 * Threshold selection (Eq. 8), the rule for contexts that grow token by token: position i of a
 * sequence becomes a nugget iff scores[i] > lambda (IEEE comparison: a NaN score never passes, -0
 * equals +0).  The number of nuggets depends on the data, so selection takes two calls with the
 * caller's read of the counts between them (one device-to-host copy; TopK needs none):
 *   dodo_count_threshold   counts[b] = number of positions of sequence b above lambda
 *   dodo_select_threshold  writes those positions, ascending, to idx[nug_off[b] .. nug_off[b+1]);
 *                          the caller lays nug_off out from the counts (a region smaller than the
 *                          count keeps the lowest positions, a larger one leaves its tail untouched)
 * The result feeds dodo_gather_kv like a TopK result.
 *   scores   [device] float[seq_off[B]]      counts [device] int32[B], written
 *   seq_off, nug_off [host] int32[B+1]       idx    [device] int32[nug_off[B]], written
 */
DODO_API int dodo_count_threshold(dodo_ctx* ctx, const float* scores, const int32_t* seq_off, int B, float lambda,
                         int32_t* counts, void* stream);
DODO_API int dodo_select_threshold(dodo_ctx* ctx, const float* scores, const int32_t* seq_off, const int32_t* nug_off,
                          int B, float lambda, int32_t* idx, void* stream);

/*
 * Lambda from sampled scores (Sec. 2.5, text after Eq. 8: the Scorer is run on sampled tokens and
 * the threshold set so that about one token in r is kept).  With k = ceil(m / r) the result is the
 * (k+1)-th largest of the m sample scores, so that exactly k of m distinct scores pass the strict
 * test; -inf when k >= m (everything must pass).  Scores rank as in dodo_select (NaN lowest; a NaN
 * result means that fewer than k+1 sample scores were numbers, and keeps nothing).
 *   sample [device] float[m], m >= 1      r >= 1      lambda [device] float[1], written
 */
DODO_API int dodo_estimate_threshold(dodo_ctx* ctx, const float* sample, int m, int r, float* lambda, void* stream);

/*
 * dodo_score followed by dodo_select in one call.  While no sequence is longer than 4096 tokens it
 * is ONE launch: the thread block that finishes a sequence's last scores runs that sequence's
 * selection; longer sequences are selected by a second launch with more threads per sequence.
 * `scores` is required (it is the hand-over buffer) and holds the same values dodo_score would
 * write; idx equals dodo_select on those values.
 */
DODO_API int dodo_score_select(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
                      const int32_t* seq_off, const int32_t* nug_off, int B, uint32_t flags,
                      float* scores, int32_t* idx, void* stream);

/*
 * Nugget gather (Eq. 5): append the selected tokens' K and V rows to each sequence's nugget cache.
 *   K, V       [device] [seq_off[B], H, dh] in `dtype` (one row per context token)
 *   idx        [device] int32[nug_off[B]] from dodo_select (sequence-local positions); any source is
 *              accepted, and an index outside [0, n_b) is never followed: that nugget's cache row and
 *              position stay as they were and DODO_DEV_BAD_INDEX is set in the device status word
 *   pos_base   [host]   int32[B]: absolute position of each sequence's token 0; the absolute
 *              position pos_base[b] + idx is recorded for the attention mask
 *   cacheK/V   [device] [cache_off[B], H, dh]; sequence b owns rows [cache_off[b], cache_off[b+1])
 *   cache_pos  [device] int32[cache_off[B]]
 *   cache_len  [host]   int32[B], in/out: rows already used -> rows used after the append
 * Row j of sequence b's selection lands in cache row cache_off[b] + cache_len[b] + j.  Rows already
 * in the cache are not touched.  Overflow of a region -> DODO_ERR_CAPACITY, nothing launched.
 */
DODO_API int dodo_gather_kv(dodo_ctx* ctx, const void* K, const void* V, int dtype, int H, int dh,
                   const int32_t* seq_off, const int32_t* idx, const int32_t* nug_off,
                   const int32_t* pos_base, int B, void* cacheK, void* cacheV, int32_t* cache_pos,
                   const int32_t* cache_off, int32_t* cache_len, void* stream);

/*
 * The whole compression step (Eq. 4-6 as the decoder uses them: Eq. 14, then Eq. 5): dodo_score_select
 * followed by dodo_gather_kv, with the same arguments and the same results in scores, idx, the cache
 * and cache_len.  With up to 64 sequences of up to 4096 tokens each the two launches overlap: the block
 * that selects a sequence raises a flag behind its indices, and the gather, launched with programmatic
 * stream serialization, copies a sequence's rows as soon as that flag is up instead of waiting for the
 * whole score launch, so the rows of sequences selected early are copied while later ones are scored.
 * Other batches run as the two calls.  The wait for a flag is bounded: a copy whose sequence's selection
 * has not appeared in time is left out and DODO_DEV_WAIT_TIMEOUT is set in the device status word (this
 * cannot happen unless a block of the score launch died).  K and V are in `dtype` like X.
 */
DODO_API int dodo_compress(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
                  const void* K, const void* V, int H, int dh, const int32_t* seq_off, const int32_t* nug_off,
                  const int32_t* pos_base, int B, uint32_t flags, float* scores, int32_t* idx, void* cacheK,
                  void* cacheV, int32_t* cache_pos, const int32_t* cache_off, int32_t* cache_len, void* stream);

/*
 * The same append for L layers that share one selection (Sec. 2.1: the indices chosen once serve
 * every layer's K/V), as one launch per 64 layers: the rows idx names are copied from each layer's
 * K[l], V[l] into that layer's cacheK[l], cacheV[l].  All layers share the layout (seq_off,
 * cache_off), the bookkeeping (cache_len, advanced once) and the positions (cache_pos, written once).
 * Equal, bit for bit, to L calls of dodo_gather_kv that each start from the same cache_len.
 *   L                  layers (0: nothing is done)
 *   K, V               [host] arrays of L device pointers, each [seq_off[B], H, dh] in `dtype`
 *   cacheK, cacheV     [host] arrays of L device pointers, each [cache_off[B], H, dh]
 *   everything else as in dodo_gather_kv; the pointer arrays are read before the call returns
 */
DODO_API int dodo_gather_kv_layers(dodo_ctx* ctx, int L, const void* const* K, const void* const* V, int dtype,
                          int H, int dh, const int32_t* seq_off, const int32_t* idx, const int32_t* nug_off,
                          const int32_t* pos_base, int B, void* const* cacheK, void* const* cacheV,
                          int32_t* cache_pos, const int32_t* cache_off, int32_t* cache_len, void* stream);

/*
 * Mean pooling of even chunks: the comparison system of Sec. 5.1 (Compressive Transformers as the paper runs
 * them: the text is cut evenly into segments and each segment's states are pooled by their mean into one).
 * Sequence b's n_b tokens are cut into k_b = ceil(n_b / r) segments of r consecutive tokens (the last one may be
 * shorter); the mean of each segment's K rows and V rows (fp32 sums in token order, one rounding to `dtype`)
 * is appended to the sequence's cache region exactly as dodo_gather_kv appends a nugget, with the position of
 * the segment's last token (a pooled state stands for everything up to there, so it becomes visible to a query
 * once the whole segment lies behind it).  dodo_attend then serves the pooled cache unchanged, at the same
 * number of states as the nugget cache at the same ratio.
 *   arguments as in dodo_gather_kv, with the ratio r >= 1 in place of idx / nug_off
 */
DODO_API int dodo_pool_kv(dodo_ctx* ctx, const void* K, const void* V, int dtype, int H, int dh,
                 const int32_t* seq_off, int r, const int32_t* pos_base, int B, void* cacheK, void* cacheV,
                 int32_t* cache_pos, const int32_t* cache_off, int32_t* cache_len, void* stream);

/* Bytes of device workspace dodo_attend needs for head size dh (a constant of the device: room for
 * the split partial results of the streaming kernel and for the partial results of units that the
 * tensor-core kernel cuts between thread blocks; about 39 MB on a 148-SM GPU).  Contents need no
 * initialisation.  With a smaller or NULL workspace dodo_attend still runs whatever needs none (key
 * lists that are not cut, and cuts whose pieces run as one thread-block cluster and merge in shared
 * memory: batches in which every sequence takes the same number of pieces, at most 8) and returns
 * DODO_ERR_CAPACITY only when a cut has to merge through the workspace. */
DODO_API size_t dodo_attend_workspace_bytes(const dodo_ctx* ctx, int dh);

/*
 * Attention over [nuggets ; local tokens] (Eq. 4; mixed resolution Eq. 9; compressor mode Eq. 13),
 * multi-head, logit = sm_scale * <q, k> (Eq. 16 with the base model's scale as an argument),
 * softmax and accumulation in fp32, output rounded once to `dtype`.
 *
 * Query i of sequence b sits at position q_pos0[b] + i.  Nugget row j carries cache_pos[...];
 * local row j of sequence b sits at loc_pos0[b] + j.  A key is visible iff its position is <= the
 * query's.  A query with no visible key gets O = 0 and lse = -inf.
 *   Q          [device] [q_off[B], H, dh]          O  [device] same shape, written
 *   q_off      [host] int32[B+1]                   q_pos0 [host] int32[B]
 *   cacheK/V, cache_pos, cache_off  as in dodo_gather_kv; cache_len [host] int32[B] rows in use
 *   locK/V     [device] [loc_rows, H, dh] uncompressed recent tokens (NULL if every loc_len = 0)
 *   loc_off    [host] int32[B] first local row of each sequence; loc_len [host] int32[B] (NULL = 0)
 *   loc_rows   total rows allocated in locK/locV (bounds the reads)
 *   lse        [device] float[q_off[B], H] natural-log sum-exp of the scaled logits, or NULL
 *   workspace  [device] at least dodo_attend_workspace_bytes(ctx, dh) bytes, 16-byte aligned
 * A sliding window kept as a ring needs no special handling while every local token is visible to
 * every query (decode): softmax does not depend on key order, so any rotation of the rows with
 * loc_pos0 = first position in the window gives the same result.
 * Stream order: the call behaves as ordinary work on `stream`, with one relaxation that lets
 * consecutive decode launches overlap.  The kernel is launched with programmatic stream
 * serialization, so its thread blocks may start while the kernel before it on the stream is still
 * finishing.  Ahead of its dependency wait it only issues cache hints (prefetch to L2, the device's
 * point of coherence, which fetch no value and stay correct whoever writes those lines meanwhile) --
 * except that it also READS rows of cacheK, cacheV and cache_pos there when the context knows that
 * nothing has written a nugget cache since its last dodo_attend: no dodo_gather_kv* call through
 * this context since then, and, under stream capture, that attend recorded in the same capture.
 * Sequences of dodo_* calls on one context therefore need no care (the first attend after a gather
 * reads everything after the wait).  A caller that writes a nugget cache by other means (its own
 * kernel, a copy, another context) between two dodo_attend calls on this context must call
 * dodo_cache_written(ctx) before the second.  Q, locK/locV, O, lse and the workspace are read and
 * written only after everything earlier on the stream has completed.
 * Supported: dh in {64, 128}; dtype in {DODO_F32, DODO_BF16}.
 */
DODO_API int dodo_attend(dodo_ctx* ctx, const void* Q, const int32_t* q_off, const int32_t* q_pos0,
                int dtype, int H, int dh, float sm_scale,
                const void* cacheK, const void* cacheV, const int32_t* cache_pos,
                const int32_t* cache_off, const int32_t* cache_len,
                const void* locK, const void* locV, const int32_t* loc_off,
                const int32_t* loc_len, const int32_t* loc_pos0, int loc_rows, int B,
                void* O, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Attention straight over the selected rows, without a nugget cache: one selection serving the layer's
 * query block in one call (Sec. 2.1; compressor mode, Eq. 13; with local tokens, Eq. 9).  Equal to
 * dodo_gather_kv into an empty cache followed by dodo_attend: sequence b's keys are the rows
 * K[seq_off[b] + idx[j]], V[...] for j in [nug_off[b], nug_off[b+1]), at positions pos_base[b] + idx[j],
 * then its local tokens.  The K and V tiles are assembled on the fly from the uncompressed arrays by
 * row-gather tensor copies, so nothing is written and read back; worth it where a cache would be used
 * once (a one-shot query over a document), not for decoding, which re-reads the cache every token.
 *   K, V      [device] [seq_off[B], H, dh] uncompressed (one row per context token), 16-byte aligned
 *   idx       [device] int32[nug_off[B]] sequence-local positions, e.g. from dodo_select; an index
 *             outside [0, n_b) is clamped into the sequence and DODO_DEV_BAD_INDEX is set
 *   seq_off, nug_off, pos_base  [host] as in dodo_gather_kv
 *   everything else as in dodo_attend (the workspace too)
 * Runs on the tensor-core kernel only: dtype DODO_BF16, dh 128, sm_scale > 0; else DODO_ERR_UNSUPPORTED.
 */
DODO_API int dodo_attend_indexed(dodo_ctx* ctx, const void* Q, const int32_t* q_off, const int32_t* q_pos0, int dtype,
                        int H, int dh, float sm_scale, const void* K, const void* V, const int32_t* seq_off,
                        const int32_t* idx, const int32_t* nug_off, const int32_t* pos_base, const void* locK,
                        const void* locV, const int32_t* loc_off, const int32_t* loc_len, const int32_t* loc_pos0,
                        int loc_rows, int B, void* O, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* Tells the context that a nugget cache was written by something other than its own dodo_gather_kv*
 * calls (see "Stream order" above): the next dodo_attend reads no cache row ahead of its dependency
 * wait.  Host-side flag only; nothing is launched. */
DODO_API int dodo_cache_written(dodo_ctx* ctx);

/*
 * The whole path for one layer on HOST buffers (Eq. 6/15 -> Eq. 14 -> Eq. 5 -> Eq. 9 per decode
 * token): uploads the batch, compresses every sequence's context (fused score + TopK with k_b =
 * nug_off[b+1] - nug_off[b], then gather into an empty nugget cache), runs `steps` decode tokens per
 * sequence, each attending its nuggets plus the `local` most recent uncompressed positions (itself
 * included), and downloads the outputs.  Everything is enqueued on `stream`; use pinned host memory
 * for the copies to be asynchronous, and synchronise the stream before reading hO or changing an
 * input.  When hK and hV are pinned and mapped for the device (cudaHostAlloc, cudaHostRegister, a
 * framework's pinned tensors) they are not uploaded: only nuggets' rows are ever needed (Eq. 5), so
 * the gather reads those rows in place over the bus, 1/r of the bytes; pageable hK/hV are uploaded
 * whole.  The results are the same either way.
 *   hX [seq_off[B], d], hw [d], hK/hV [seq_off[B], H, dh]           [host] context
 *   hLocK/hLocV [B, local + steps, H, dh]  [host] uncompressed tokens after each context: `local`
 *               seed tokens, then the decoded tokens' K/V rows, at positions n_b, n_b + 1, ...
 *   hQ [steps, B, H, dh]  [host] decode queries; token t of sequence b sits at n_b + local + t
 *   hO [steps, B, H, dh]  [host] written
 *   arena  [device] scratch of at least dodo_host_arena_bytes(...) bytes, 256-byte aligned
 * At most 64 sequences per call.
 */
DODO_API size_t dodo_host_arena_bytes(const dodo_ctx* ctx, int dtype, int d, int H, int dh, int total_tokens,
                                      int total_nuggets, int B, int local, int steps);
DODO_API int dodo_compress_decode_host(dodo_ctx* ctx, const void* hX, const void* hw, const void* hK, const void* hV,
                                       int dtype, int d, int H, int dh, const int32_t* seq_off,
                                       const int32_t* nug_off, int B, const void* hLocK, const void* hLocV,
                                       int local, const void* hQ, int steps, float sm_scale, void* hO,
                                       void* arena, size_t arena_bytes, void* stream);

/*
 * dodo_attend for callers that must not allocate.  (The paper has no counterpart to this entry
 * point: it computes exactly what dodo_attend computes and exists only for deployment reasons.)
 *
 * Who needs it: code that is handed device pointers and a stream but may not call cudaMalloc --
 * for example a plug-in inside a serving engine whose memory pool already owns the whole device, or
 * a latency-critical path that cannot afford the device-wide synchronisation cudaMalloc and
 * cudaFree imply.  Such callers can create neither a dodo_ctx (dodo_create allocates its counters)
 * nor a workspace.  This function therefore takes no context and no workspace: its split-K
 * partial results and arrival counters live in a fixed 4 MiB device array inside the library
 * image, which every GPU that loads the library holds until the process exits.  The call makes no
 * device or host allocation.
 *
 * Arguments are those of dodo_attend without ctx/workspace; `err` (may be NULL) receives the reason
 * of a failure, up to err_len bytes.  The CUDA device that is current when the call is made is used.
 * Limits: at most 64 sequences per call, and the split-K plan must fit the fixed array.  A plan
 * writes at most 16 x 2 x SMs partial rows of (dh + 2) floats -- 2.5 MB at head size 128 on 148 SMs
 * -- so on devices of up to about 250 SMs the second limit is never met.  Beyond either limit the
 * call returns DODO_ERR_CAPACITY and launches nothing -- use dodo_attend with a workspace instead.
 * The first call on each device looks up the array's device address (host threads may make first
 * calls concurrently: the look-up is done under a lock); make that first call outside any stream
 * capture.
 * All calls share the one array, which still holds the previous call's contents (the counters are
 * re-zeroed on `stream` at the start of each call).  Calls that overlap on the GPU -- two streams,
 * or two host threads without ordering -- race on it and produce wrong results: keep calls to this
 * function ordered per device.  Results can differ from dodo_attend's in the last fp32 bits because
 * the keys may be split differently.  There is no device status to read: the kernel this function
 * launches has no bounded wait and follows no caller-supplied index, so it cannot report anything.
 * No cache row is read ahead of the launch's dependency wait (the function cannot know what precedes it).
 */
DODO_API int dodo_attend_noalloc(const void* Q, const int32_t* q_off, const int32_t* q_pos0, int dtype, int H,
                                 int dh, float sm_scale, const void* cacheK, const void* cacheV,
                                 const int32_t* cache_pos, const int32_t* cache_off, const int32_t* cache_len,
                                 const void* locK, const void* locV, const int32_t* loc_off,
                                 const int32_t* loc_len, const int32_t* loc_pos0, int loc_rows, int B, void* O,
                                 float* lse, void* stream, char* err, size_t err_len);

#ifdef __cplusplus
}
#endif
#endif /* DODO_H */
