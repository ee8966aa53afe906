/*
 * libh1b -- decode-time attention read directly from a hybrid compressed KV
 * cache (H1B-KV): every cached key is an m-bit sign sketch sign(R k) of a fixed
 * Gaussian projection (Section IV-A, Eq. 2), every cached value is a vector of
 * 4-bit codes with a scale and a zero-point (Section IV-B, Eq. 4), scores are
 * normalised Hamming inner products (Eq. 3) and the output is
 * softmax(alpha/tau) * V_dequant (Section IV-C, Eq. 5).
 *
 * C ABI, CUDA (sm_100a) behind it.  No C++ or framework types cross this
 * boundary: plain pointers, marked HOST or DEVICE, and sizes.
 *
 * Conventions
 *   - Every call returns 0 (H1B_OK) or a negative H1B_ERR_* code; the text of
 *     the last error of a context is h1b_last_error().  Nothing aborts or
 *     throws.  Argument errors are detected on the host before any launch, so
 *     a failed call has written nothing.
 *   - Ownership: the library owns only the host-side context.  The caller
 *     allocates the device workspace (h1b_cache_bytes() bytes, 256-byte
 *     aligned) and every input/output buffer, and keeps them alive until the
 *     stream work that uses them has completed.  h1b_free() does not free the
 *     workspace.
 *   - Asynchrony: h1b_append_kv() and h1b_decode_attention() only enqueue work
 *     on `stream` (a cudaStream_t passed as void*, NULL = the default stream).
 *     Use one stream at a time per context.  Contexts may be created and
 *     used from several host threads (one thread at a time per context): the
 *     per-device set-up the library keeps (kernel attributes, the address of
 *     its built-in scratch array) is made under a lock, in h1b_init_projection().
 *   - Symbols: d = head_dim, m = sketch_bits (the paper's b), G = group_size,
 *     L = n_layers, Hq / Hkv = query / KV heads, B = sequences in the call.
 *     The projection is held as Rt[d][m] (row-major), Rt[i][j] = R[j][i] for
 *     the paper's R in R^{m x d}; one matrix per layer, shared by all heads and
 *     by keys and queries.
 *   - Sketch bit j of a vector x is 1 iff sum_i x_i * Rt[i][j] >= 0 (s_j = +1).
 *   - Values: per token, per KV head, per group of G consecutive channels:
 *     scale = fp16((max - min)/15), zero = min, code = clamp(rne((v - zero)/scale), 0, 15),
 *     code = 0 when scale == 0.  Dequantised value = code * scale + zero.
 *   - Score of token t for a query: m - 2 * popcount(s_q xor s_t); alpha = score / m.
 *     All cached tokens [0, len) are attended, the one just appended included.
 *     Query head h reads KV head h / (Hq / Hkv).  An empty sequence gives zeros.
 *   - d = 64 (the paper's 60M model: 12 layers, 8 heads of 64 channels) runs
 *     through the same 128-channel kernels, two KV heads per cache slab; nothing
 *     of that shows at this interface (shapes, exports and results are per
 *     head), except the restrictions listed at h1b_config.head_dim.
 *   - With H1B_FLAG_FP16_VALUES (the "1-bit keys only" row of the ablation,
 *     Table V) values are cached as the fp16 numbers they arrive as: no codes,
 *     scales or zero-points; the output is softmax(alpha/tau) * V.
 */
#ifndef H1B_H
#define H1B_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define H1B_OK               0
#define H1B_ERR_INVALID_ARG (-1)  /* a size, index or flag is out of range            */
#define H1B_ERR_NULL        (-2)  /* a required pointer is NULL                        */
#define H1B_ERR_UNSUPPORTED (-3)  /* valid in principle, no kernel for this shape      */
#define H1B_ERR_CAPACITY    (-4)  /* len + n_new > max_seq for some sequence           */
#define H1B_ERR_WORKSPACE   (-5)  /* workspace too small or misaligned                 */
#define H1B_ERR_CUDA        (-6)  /* a CUDA runtime call failed (text in last_error)   */
#define H1B_ERR_TIMEOUT     (-7)  /* a bounded device-side wait gave up (poll_status)  */
#define H1B_ERR_BOUNDS      (-8)  /* bounds-checked build only: a kernel's index check
                                     failed and its access was skipped (poll_status)   */

typedef struct h1b_ctx h1b_ctx;   /* opaque, host-side */

typedef struct {
    int32_t n_layers;      /* L >= 1                                                   */
    int32_t n_q_heads;     /* Hq; a multiple of Hkv, Hq / Hkv <= 16                    */
    int32_t n_kv_heads;    /* Hkv                                                      */
    int32_t head_dim;      /* d: 128, or 64 (then Hkv even, G = 32, m <= 256)           */
    int32_t sketch_bits;   /* m: 64, 128, 256 or 512                                   */
    int32_t group_size;    /* G: 32, or 128 (= d: one scale and zero per value vector)  */
    int32_t max_batch;     /* sequences the cache can hold (<= 256)                    */
    int32_t max_seq;       /* tokens per sequence the cache can hold                   */
    int32_t device;        /* CUDA device ordinal                                      */
    uint32_t flags;        /* H1B_FLAG_* bits; every other bit must be 0               */
    int32_t page_tokens;   /* 0: one contiguous slab per sequence; > 0 (a multiple of
                              32): paged cache, tokens per page                        */
    int32_t n_pages;       /* paged cache: pages in each layer's pool (else 0)         */
} h1b_config;

/* Keep values in fp16 (keys are still 1-bit sketches); group_size must still be a
 * supported value but is not used. */
#define H1B_FLAG_FP16_VALUES 1u

/* Rotary position embedding fused into the path (not a step of the paper's
 * method: the rotation belongs to the model, and a Llama-style model caches
 * the rotated keys; fusing it saves the model a pass over K and q). With this
 * flag the key rows of an append are rotated at their cache positions and the
 * query rows of a decode call at the position of their token (the sequence's
 * last, or with Tq query tokens its last Tq) before Eq. 2; values are not
 * touched. Pairs are (channel i, channel i + d/2) of a head:
 *     x_i' = x_i c - x_{i+d/2} s,   x_{i+d/2}' = x_{i+d/2} c + x_i s,
 * (c, s) = table[position][i]. Each product and the sum are rounded to fp32
 * (no fused multiply-add) and the result once to fp16, to nearest even: the
 * rotated row is the same fp16 bits in every kernel.
 * h1b_set_rope_table must be called before the first append or decode. */
#define H1B_FLAG_ROPE 2u

/* Bytes of one cached token of one KV head: m/8 + d/2 + (d/G)*4 (Section IV-B
 * storage statement plus the fp16 scale and zero per group); m/8 + 2d with
 * H1B_FLAG_FP16_VALUES. 0 if invalid. */
size_t h1b_entry_bytes(const h1b_config *cfg /* HOST */);

/* Paged cache (page_tokens > 0; not a step of the paper's method: the cache
 * layout serving systems use for ragged batches). A page holds page_tokens
 * consecutive tokens of every KV head of one layer; each layer has its own pool
 * of n_pages pages; ONE block table per sequence, shared by all layers and
 * heads, names the pool page that holds tokens [k * page_tokens, (k+1) *
 * page_tokens) of the sequence. max_seq bounds a sequence's table, the pool
 * bounds the total. A new context has empty tables: give every sequence its
 * pages with h1b_set_block_table() before appending to it.
 *
 * h1b_set_block_table: sequence `seq` owns pages_host[0 .. n) (HOST int32, each
 * in [0, n_pages), n * page_tokens <= max_seq rounded up to whole pages), in
 * this order. May grow or shrink a table between steps; entries that cover
 * cached tokens must keep their pages. Stream-ordered like the other calls.
 * H1B_ERR_INVALID_ARG on a contiguous cache, on bad page numbers, on a page
 * that is listed twice or that another sequence's table holds, or when fewer
 * pages than the sequence's cached tokens need. */
int h1b_set_block_table(h1b_ctx *ctx, int seq, const int32_t *pages_host, int n, void *stream);

/* Rotary table (H1B_FLAG_ROPE): cos_sin_host is HOST fp32 [n_positions][d/2][2],
 * (cos, sin) of the angle of pair i at each position, copied into the workspace
 * (synchronous: returns when the copy is done). n_positions >= 1; positions
 * from max_seq (rounded up to 32) on are not kept. A call that would reach a position the table does not hold
 * fails with H1B_ERR_CAPACITY (a replayed graph: the position is clamped to the
 * table's last). H1B_ERR_INVALID_ARG if the cache was made without the flag. */
int h1b_set_rope_table(h1b_ctx *ctx, const float *cos_sin_host, int n_positions, void *stream);

/* Bytes of device workspace the caller must provide for this configuration
 * (projection matrices, lengths, split-K scratch, staging and the packed cache
 * itself). 0 if the configuration is invalid or unsupported. */
size_t h1b_cache_bytes(const h1b_config *cfg /* HOST */);

/* Create a context over a caller-owned workspace and install the projection
 * matrices (Section IV-A: "a fixed, pre-generated Gaussian matrix").
 *   seed       used only when Rt_host is NULL
 *   Rt_host    HOST, nullable: float32 [L][d][m]; NULL = draw N(0,1) from `seed`
 *              on the host (Box-Muller over a splitmix64 counter stream)
 *   workspace  DEVICE, 256-byte aligned, workspace_bytes >= h1b_cache_bytes(cfg)
 *   out        HOST: receives the context
 * Zero-fills the workspace, copies Rt to the device, sets all lengths to 0 and
 * synchronises the stream before returning. */
int h1b_init_projection(const h1b_config *cfg, uint64_t seed, const float *Rt_host,
                        void *workspace, size_t workspace_bytes, void *stream,
                        h1b_ctx **out);

/* Compress and append new key/value rows (Eq. 2 on keys, Eq. 4 on values).
 *   k, v        DEVICE: fp16 [n_layers][B][Tn][Hkv][d]
 *   n_new_host  HOST, nullable: int32 [B], 0 <= n_new[b] <= Tn rows of sequence b
 *               are appended (the first n_new[b] of its Tn); NULL = Tn for all
 * Sequence b of the call is sequence b of the cache.  Row tn of sequence b goes
 * to position len[layer][b] + tn; afterwards len[layer][b] += n_new[b].
 * H1B_ERR_CAPACITY (nothing written) if any sequence would exceed max_seq or,
 * with a paged cache, the pages its block table holds.
 * Every DEVICE tensor of this interface (k, v, q, out) must start on a 16-byte
 * boundary: H1B_ERR_INVALID_ARG otherwise, before anything is launched. */
int h1b_append_kv(h1b_ctx *ctx, int layer_begin, int n_layers, const void *k, const void *v,
                  const int32_t *n_new_host, int B, int Tn, void *stream);

/* One decode step of attention over the compressed cache (Eq. 3 and Eq. 5):
 * sketch the queries, score every cached token by popcount, softmax with
 * temperature tau, weight the dequantised values.
 *   q        DEVICE: fp16 [n_layers][B][Hq][d]
 *   inv_tau  1/tau, finite and > 0
 *   out      DEVICE: float32 [n_layers][B][Hq][d]
 * Uses the split-K scratch inside the workspace: calls on one context must not
 * overlap on the GPU. */
int h1b_decode_attention(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q,
                         float inv_tau, void *out, int B, void *stream);

/* Decode attention for the last Tq tokens of every sequence at once (chunked
 * prefill, verification of speculated tokens). The Tq query tokens are the
 * sequence's last Tq cached tokens, already appended: query token i
 * (0 <= i < Tq) attends to cached tokens [0, len - Tq + i + 1), i.e. to
 * everything up to and including itself (Eq. 3 and Eq. 5 per query token).
 * The paper describes one query per step; this is the same computation for
 * several queries that share every cache tile they read.
 *   q    DEVICE: fp16 [n_layers][B][Tq][Hq][d]      1 <= Tq <= H1B_MAX_QUERY_TOKENS
 *   out  DEVICE: float32 [n_layers][B][Tq][Hq][d]
 * H1B_ERR_INVALID_ARG if some sequence of the call holds fewer than Tq tokens.
 * Tq = 1 is h1b_decode_attention(). The split-K scratch of the workspace is
 * sized for the largest call this allows (max_batch sequences, Tq = 16), so no
 * valid call runs out of it. */
#define H1B_MAX_QUERY_TOKENS 16
int h1b_decode_attention_multi(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, int Tq,
                               float inv_tau, void *out, int B, void *stream);

/* Attention for a whole run of Tn query tokens per sequence (a prompt, or a
 * chunk of one): the queries are the sequences' last Tn cached tokens (append
 * their keys and values first), query token i attends to cached tokens
 * [0, len - Tn + i + 1). Any Tn >= 1. Runs of 32 tokens or more (head
 * dimension 128) are processed in blocks of 128 query
 * tokens x 64 cached tokens on the tensor cores: Eq. 3 as one dense +-1
 * contraction per block (exact integers), Eq. 5 with each tile's values
 * dequantised once for all its queries; `out` doubles as scratch for the query
 * sketches until its rows are written. Other runs walk in blocks of
 * H1B_MAX_QUERY_TOKENS query tokens, each block one pass of the decode kernels
 * over the part of the cache it may see. q: DEVICE fp16 [n_layers][B][Tn][Hq][d];
 * out: DEVICE float32, same shape. Every sequence must hold at least Tn
 * tokens in every layer of the call (H1B_ERR_INVALID_ARG otherwise). With the
 * rotary option each query is rotated at the position of its token. */
int h1b_prefill_attention(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q, int Tn,
                          float inv_tau, void *out, int B, void *stream);

/* One whole decode step on device tensors, all L layers: append one new token per
 * sequence (Eq. 2, Eq. 4) and run decode attention over the grown cache (Eq. 3,
 * Eq. 5). Same result as h1b_append_kv(Tn = 1) followed by h1b_decode_attention(),
 * in three kernel launches instead of four.
 *   k, v  DEVICE: fp16 [L][B][1][Hkv][d]      q  DEVICE: fp16 [L][B][Hq][d]
 *   out   DEVICE: float32 [L][B][Hq][d] */
int h1b_decode_step(h1b_ctx *ctx, const void *k, const void *v, const void *q, float inv_tau,
                    void *out, int B, void *stream);

/* The same for layers [layer_begin, layer_begin + n_layers) only: what a model
 * that runs its layers one after the other calls once per layer.
 *   k, v  DEVICE: fp16 [n_layers][B][1][Hkv][d]   q  DEVICE: fp16 [n_layers][B][Hq][d]
 *   out   DEVICE: float32 [n_layers][B][Hq][d] */
int h1b_decode_step_layers(h1b_ctx *ctx, int layer_begin, int n_layers, const void *k,
                           const void *v, const void *q, float inv_tau, void *out, int B,
                           void *stream);

/* Stream capture. h1b_append_kv(), h1b_decode_attention(), h1b_decode_step() and
 * h1b_decode_step_layers() only enqueue kernels, so they may be recorded into a
 * CUDA graph; nothing has to be called first (every kernel attribute a context
 * can need is set when the context is created). The kernels read the sequence
 * lengths from device memory,
 * so every replay appends at, and attends up to, the then-current end of each
 * sequence. Frozen at capture time: the pointers, B, n_new and the number of
 * splits per sequence (which chunks a split takes is worked out on the device
 * from the length at that moment, so growth is covered). The host's copy of
 * the lengths only sees the captured calls, not their replays: call
 * h1b_sync_lengths() after replaying and before any other call on the context.
 * A replay that finds a sequence full writes nothing for it, leaves its length
 * alone and raises H1B_ERR_CAPACITY at the next h1b_poll_status().
 *
 * h1b_sync_lengths: copy the device's lengths into the host's copy; synchronises
 * `stream`. */
int h1b_sync_lengths(h1b_ctx *ctx, void *stream);

/* h1b_decode_attention() for callers that must not allocate and cannot spare
 * scratch of their own. (No counterpart in the paper: this is a deployment
 * convenience, not a step of the method.)
 *
 * Who this is for: code that runs after its process has handed all device
 * memory to a fixed arena, a plug-in inside another runtime's region where
 * cudaMalloc/cudaFree (and anything that calls them, a tensor library's
 * allocator included) is forbidden or would synchronise the device, or a
 * latency-critical loop that may not take the allocator's lock. Such callers
 * still own the cache, q and out; what they lack is a place for this call's
 * temporaries. Here the temporaries (the query sketches and the split-K
 * partial results) live in an 8 MiB array built into the library image, so the
 * call allocates nothing, frees nothing and writes nothing in the workspace's
 * scratch region. Every device that loads the library holds those 8 MiB until
 * the process exits.
 *
 * Same arguments, same result and same errors as h1b_decode_attention(), plus:
 *   - H1B_ERR_CAPACITY, with the needed and the available byte counts in
 *     h1b_last_error(), when ONE layer of the call does not fit with one split
 *     per sequence:
 *         B * Hkv * ceil(g / k) * k * 528 bytes of partials, g = Hq / Hkv and
 *         k = g for g <= 2, else 4 (heads go through in groups of four); with
 *         d = 64, two KV heads share a cache slab: Hkv / 2 * ceil(2g / k) * k
 *         with k = 2 for g = 1, else 8
 *     plus L * max_batch * Hq * m/8 bytes of sketches (all layers and sequences
 *     of the context, rounded up to 256) must be <= 8 MiB (8 388 608). A call
 *     with more layers than fit at once sends them through the array in passes,
 *     and fewer splits per sequence are used than the automatic choice when
 *     those would not fit (slower, same result up to summation order).
 *   - the context's device must be the current device.
 *   - nothing is looked up or set up by the call itself: the array's device
 *     address was obtained (cudaGetSymbolAddress) when the first context on
 *     this device was created, in h1b_init_projection(), which also loaded
 *     the kernels it launches. From its first use the call is therefore only
 *     kernel launches; create the context outside any region in which
 *     allocation is forbidden, and outside any stream capture.
 * All contexts and all calls in the process share the one array per device, and
 * it keeps whatever the last call left in it; nothing in it has to be
 * initialised, since a call reads only what it has written itself. Two calls
 * whose kernels overlap on the GPU (different streams, different contexts)
 * race on it: order them on one stream or with events. */
int h1b_decode_attention_static(h1b_ctx *ctx, int layer_begin, int n_layers, const void *q,
                                float inv_tau, void *out, int B, void *stream);

/* The same step for callers whose tensors live in host memory: copies k, v, q
 * (HOST, fp16, [L][B][1][Hkv][d], [L][B][1][Hkv][d], [L][B][Hq][d]; pinned
 * memory makes the copies asynchronous) into staging inside the workspace,
 * appends one token per sequence to all L layers, runs decode attention over
 * all layers, copies the result to out (HOST, float32 [L][B][Hq][d]) and
 * synchronises the stream. When k, v and q lie back to back in host memory (in
 * that order) they travel in one copy. */
int h1b_decode_step_host(h1b_ctx *ctx, const void *k_host, const void *v_host,
                         const void *q_host, float inv_tau, void *out_host, int B,
                         void *stream);

/* Synchronise the context's device and release the host-side context. The
 * workspace stays with the caller. */
int h1b_free(h1b_ctx *ctx);

/* ---- introspection and test helpers (synchronous) ------------------------ */

/* Copy layer `layer`'s projection to Rt_host (HOST float32 [d][m]). */
int h1b_get_projection(h1b_ctx *ctx, int layer, float *Rt_host);

/* Copy layer `layer`'s lengths to len_host (HOST int32 [max_batch]); also
 * checks them against the host mirror (H1B_ERR_INVALID_ARG on mismatch). */
int h1b_get_lengths(h1b_ctx *ctx, int layer, int32_t *len_host);

/* Forget the cached tokens of sequence `seq` in all layers (-1 = all
 * sequences): lengths become 0; the bytes are not cleared. */
int h1b_reset(h1b_ctx *ctx, int seq);

/* Set the length of sequence `seq` (-1 = all) in all layers to new_len, which
 * must not exceed any of their current lengths (roll back the last tokens). */
int h1b_truncate(h1b_ctx *ctx, int seq, int new_len);

/* The same, ordered on `stream` instead of waiting for the device (rejecting
 * speculated tokens between two decode steps): the caller keeps every call that
 * touches this cache on that one stream, or orders them with events. Both
 * h1b_reset and h1b_truncate wait for the whole device before and after. */
int h1b_truncate_async(h1b_ctx *ctx, int seq, int new_len, void *stream);

/* Unpack cached tokens [t0, t0+n) of (layer, seq, kv_head) into a canonical
 * layout, independent of the packed device layout (all HOST, any may be NULL):
 *   words  uint32 [n][m/32]: sketch bit j is bit (j % 32) of word j / 32
 *   codes  uint8  [n][d]:    one 4-bit code per byte
 *   scale, zero  uint16 [n][d/G]: fp16 bit patterns
 * With H1B_FLAG_FP16_VALUES only `words` exists: codes, scale and zero must be
 * NULL (H1B_ERR_INVALID_ARG otherwise); see h1b_export_values(). */
int h1b_export_cache(h1b_ctx *ctx, int layer, int seq, int kv_head, int t0, int n,
                     uint32_t *words, uint8_t *codes, uint16_t *scale, uint16_t *zero);

/* H1B_FLAG_FP16_VALUES only (H1B_ERR_INVALID_ARG otherwise): the cached values
 * of tokens [t0, t0+n) of (layer, seq, kv_head).
 *   values  HOST: uint16 [n][d], fp16 bit patterns, channel-contiguous */
int h1b_export_values(h1b_ctx *ctx, int layer, int seq, int kv_head, int t0, int n,
                      uint16_t *values);

/* Sketch one query (DEVICE fp16 [d]) with layer `layer`'s projection and score
 * it against every cached token of (layer, seq, kv_head):
 *   qwords_host  HOST, nullable: uint32 [m/32]
 *   score_host   HOST, nullable: int32 [len] = m - 2 * Hamming */
int h1b_debug_scores(h1b_ctx *ctx, int layer, int seq, int kv_head, const void *q,
                     uint32_t *qwords_host, int32_t *score_host);

/* After an attention call (any of the decode / multi / prefill-attention / static
 * entry points) has completed: what the attention kernel itself wrote for one
 * (layer, sequence, query token, query head) of that call's LAST launch, split by
 * split (HOST outputs, room for max_splits entries each):
 *   n_splits_host  the number S of splits the sequence was dealt into
 *   hmin_host[s]   the smallest Hamming distance (Eq. 3) split s saw among the
 *                  tokens this head attends to, as a float; 1048576 if it saw none
 *   wsum_host[s]   sum over those tokens of 2^((hmin[s] - Hamming_t) * c),
 *                  c = 2 log2(e) / (m tau): the split's softmax denominator (Eq. 5)
 * Split s covers chunks [s*q + min(s, r), (s+1)*q + min(s+1, r)) of the C =
 * ceil(len / 32) chunks of 32 tokens the sequence holds, q = C / S, r = C mod S.
 * A test compares these with a CPU statement of Eq. 3, so the scoring inside the
 * production kernel is checked bit for bit and not only through the outputs.
 * H1B_ERR_INVALID_ARG when the indices are not part of that launch. */
int h1b_debug_partials(h1b_ctx *ctx, int layer, int seq, int q_token, int q_head,
                       int32_t *n_splits_host, float *hmin_host, float *wsum_host, int max_splits);

/* Test helpers of h1b_prefill_attention (no counterpart in the paper).
 *   h1b_debug_prompt_scores  the NEXT h1b_prefill_attention call that takes the tile route also writes the integer
 *                            scores m - 2 * Hamming (Eq. 3) its tensor-core contraction produced for one (layer,
 *                            sequence, query head) to score_dev, DEVICE int32 [Tn][n_tokens] (entry [i][t] for query
 *                            token i of the run and cached token t < n_tokens; tokens beyond the tiles that query
 *                            block visits are not written). score_dev NULL switches it off.
 *   h1b_debug_prompt_route   tiles = 0: h1b_prefill_attention walks every run in blocks of H1B_MAX_QUERY_TOKENS through
 *                            the decode kernels (the route short runs take); tiles = 1 (default): runs of 32 query tokens
 *                            or more take the 128 x 64 tile kernel where the cache format allows it (head dimension
 *                            128). Both routes compute the same thing. */
int h1b_debug_prompt_scores(h1b_ctx *ctx, int layer, int seq, int q_head, int32_t *score_dev, int n_tokens);
int h1b_debug_prompt_route(h1b_ctx *ctx, int tiles);
/*   h1b_debug_prompt_stall   the failure path of the tile kernel, exercised without harming anything: in the NEXT
 *                            h1b_prefill_attention call that takes the tile route, the warp that requests the copies
 *                            and issues the contractions stays idle and every wait is limited to limit_ns (1 .. 1e9).
 *                            The row threads' first wait runs out; they record the time-out in the device status word,
 *                            the block releases its tensor memory and the kernel returns normally. That call's output
 *                            is undefined; h1b_poll_status() then reports H1B_ERR_TIMEOUT once, and the context keeps
 *                            working. H1B_ERR_INVALID_ARG for a limit outside the range. */
int h1b_debug_prompt_stall(h1b_ctx *ctx, uint64_t limit_ns);

/* Bounds-checked build (no counterpart in the paper; a debugging aid). When the
 * library is compiled with -DH1B_DEBUG_BOUNDS, every address a kernel derives
 * from its parameters for global memory (cache chunks, split-K partials, query
 * sketches) and every carve of its shared memory is range-checked before use; a
 * failing check records its number in the device status word and the access is
 * skipped (nothing traps or faults), and h1b_poll_status() then returns
 * H1B_ERR_BOUNDS once. The ordinary build contains none of this.
 *   h1b_bounds_checked       1 if this library has the checks, else 0
 *   h1b_debug_bounds_probe   launches a kernel whose one check fails on purpose
 *                            and verifies that its guarded store was not made;
 *                            the next h1b_poll_status() reports H1B_ERR_BOUNDS.
 *                            H1B_ERR_UNSUPPORTED in the ordinary build.
 *                            Synchronises `stream`. */
int h1b_bounds_checked(void);
int h1b_debug_bounds_probe(h1b_ctx *ctx, void *stream);

/* Failure-path probe (no counterpart in the paper). Launches one warp that waits
 * for at most limit_ns nanoseconds (1 .. 1e9) on a barrier phase nothing will
 * complete, with the same bounded wait the attention and long-append kernels
 * use for their copies and tensor-core work. The wait runs out, the warp
 * records the time-out in the device status word and the kernel returns
 * normally: nothing traps, faults or spins on. After the stream has been
 * synchronised h1b_poll_status() then returns H1B_ERR_TIMEOUT once and H1B_OK
 * afterwards, and the context stays usable. Asynchronous on `stream`. */
int h1b_debug_wait_timeout(h1b_ctx *ctx, uint64_t limit_ns, void *stream);

/* Force the number of sequence splits of the decode kernel (0 = automatic).
 * H1B_ERR_INVALID_ARG if the split-K scratch cannot hold that many. */
int h1b_set_splits(h1b_ctx *ctx, int splits);

/* After the stream has been synchronised: 0, H1B_ERR_TIMEOUT if a kernel gave
 * up a bounded wait since the last poll, H1B_ERR_CAPACITY if a replayed append
 * found a sequence full, or (bounds-checked build) H1B_ERR_BOUNDS if a kernel's
 * index check failed (the flag is cleared). */
int h1b_poll_status(h1b_ctx *ctx);

/* Time the dominant kernel. While enabled, every h1b_decode_attention() brackets
 * the launch of its split-K attention kernel with a pair of CUDA events on the
 * call's stream (at most 4096 pairs between two reads; later launches are not
 * recorded). Events are created on the first enabling call. */
int h1b_set_profiling(h1b_ctx *ctx, int enable);

/* Synchronise the device, return the summed duration (milliseconds) and the
 * number of the recorded kernel launches (both HOST), and forget them. */
int h1b_read_profile(h1b_ctx *ctx, double *decode_ms, int64_t *decode_launches);

/* Kernel launches enqueued by this context so far. */
int64_t h1b_launch_count(const h1b_ctx *ctx);

/* Text of the last error recorded on this context ("" if none). With ctx ==
 * NULL: the text of the last failed h1b_init_projection() on this thread. */
const char *h1b_last_error(const h1b_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* H1B_H */
