/*
 * echokv.h -- C-ABI of the B200 (sm_100a) EchoKV decode-attention library.
 *
 * What the library computes (paper, Section 3.2 "Network Architecture" and Eq. 6-7):
 * the layers of a model are split into groups of S; the first layer of a group
 * (the "anchor", Eq. 1) keeps its whole KV cache, every other layer keeps only the
 * first m = r * head_dim flattened dims of each token's K and V (Eq. 2).  At decode
 * time the dropped dims of a compressed layer are predicted per token by one linear
 * map per layer and per kind (K, V),
 *     C_hat_drop[t] = W [C_anchor[t] ; C_local[t]]                         (Eq. 3)
 * the cache is rebuilt as Reshape([C_local ; C_hat_drop]) (Eq. 6) and fed to
 *     out_h = softmax_t(q_h . K~[t, kv(h)] * scale) V~[:, kv(h)]           (Eq. 7)
 * with kv(h) = h / (n_q_heads / n_kv_heads).  The reconstructed K~/V~ exist only
 * on chip; they are never written to device memory.
 *
 * Conventions
 *  - Every function returns an int status (ECHOKV_OK = 0, negative = error) and
 *    never throws, aborts or traps.  echokv_strerror() names a status.
 *  - "device pointer" = memory of the CUDA device named in the config, allocated by
 *    the caller (e.g. by PyTorch); the library BORROWS it: it must stay valid until
 *    echokv_destroy().  "host pointer" = ordinary host memory, read during the call
 *    only, unless stated otherwise.  The library itself allocates no device memory.
 *  - Alignment: pools, predictors, queries (q), new K / V rows (k_new, v_new), side buffers, scratch and
 *    result buffers (out) must be 16-byte aligned -- the kernels move them 16 bytes at a time; workspaces
 *    256-byte aligned.  A pointer aligned to less is refused with ECHOKV_EINVAL on the host, before any launch.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *    that take a stream only enqueue work on it and return; the *_host calls and
 *    echokv_get_device_status() synchronise.
 *  - Flattened KV index = kv_head * head_dim + feature.  Retained heads are heads
 *    0 .. r-1.  Storage type (cache, weights, queries, new K/V) is the config's
 *    dtype; accumulation is always fp32; outputs are fp32.
 *  - Page pools: layer l's K pool and V pool are each
 *        [n_pages][page_tokens][width(l)]   row-major, width = D for an anchor
 *        layer, m for a compressed layer (no pool when m = 0),
 *    and one int32 block table [max_batch][max_pages_per_seq], shared by all layers,
 *    maps (sequence slot, token / page_tokens) to a page id in [0, n_pages).
 *  - Predictors: Wk, Wv are [D - m][D + m] row-major; column i < D multiplies anchor
 *    dim i, column D + i multiplies local dim i; row j produces flat dim m + j.
 */
#ifndef ECHOKV_H
#define ECHOKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct echokv_ctx echokv_ctx;

enum { ECHOKV_BF16 = 0, ECHOKV_FP32 = 1 };

enum {
  ECHOKV_OK = 0,
  ECHOKV_EINVAL = -1,         /* NULL pointer, bad dimension, layer out of range          */
  ECHOKV_ENOTANCHOR = -2,     /* echokv_full_attention on a layer that keeps only m dims   */
  ECHOKV_ENOTCOMPRESSED = -3, /* echokv_set_weights on an anchor layer                     */
  ECHOKV_ECAPACITY = -4,      /* batch > max_batch, workspace too small, length > pages    */
  ECHOKV_ENOWEIGHTS = -5,     /* decode on a compressed layer before echokv_set_weights    */
  ECHOKV_ECUDA = -6,          /* a CUDA runtime / driver call failed                       */
  ECHOKV_ETIMEOUT = -7,       /* device status: a bounded on-chip wait ran out             */
  ECHOKV_EBADPAGE = -8,       /* device status: page id or sequence slot out of range      */
  ECHOKV_EUNSUPPORTED = -9,   /* shape outside what the kernels handle                     */
  ECHOKV_ENOTABLE = -10,      /* a call that needs the block table before it was set       */
  ECHOKV_EBADLENGTH = -11,    /* device status: a sequence length < 1 or beyond capacity   */
  ECHOKV_ESCRATCH = -12       /* problem too large for the fixed scratch of the no-alloc entry */
};

typedef struct {
  int32_t n_layers;
  int32_t n_q_heads;
  int32_t n_kv_heads;        /* must divide n_q_heads                                      */
  int32_t head_dim;          /* 64 or 128                                                  */
  int32_t group_size;        /* S >= 1; layer l is an anchor iff l % S == 0 (Eq. 1)        */
  int32_t n_retained_heads;  /* r in [0, n_kv_heads]; m = r * head_dim (Eq. 2)             */
  int32_t page_tokens;       /* tokens per page: 16, 32, 64 or 128                         */
  int32_t max_batch;         /* rows of the block table                                    */
  int32_t max_pages_per_seq; /* columns of the block table                                 */
  int32_t dtype;             /* ECHOKV_BF16 or ECHOKV_FP32                                 */
  int64_t n_pages;           /* pages per pool                                             */
  float softmax_scale;       /* 0 -> 1 / sqrt(head_dim) (Eq. 7)                            */
  int32_t device;            /* CUDA device ordinal                                        */
  int32_t n_retained_dims;   /* 0: m = n_retained_heads * head_dim.  Otherwise m itself, in flat dims: a
                                multiple of 64 in [0, D] that need not end on a head boundary (the paper's
                                m = 64 keeps half of head 0, its m = 384 three heads); n_retained_heads is then
                                ignored.  Eq. 6 concatenates at the flat index m: of a head that m splits the
                                dims below m are the stored ones and the rest are predicted.  The kernels that
                                work on whole heads predict such a head whole, with `m mod head_dim` one-hot rows
                                in front of the predictors that pass its stored dims through unchanged (exact);
                                the extended predictors live in the workspace (echokv_query_sizes accounts for
                                them) and echokv_set_weights builds them */
  int32_t save_k;            /* non-zero: the "save K" setting of Section 5.2 -- compressed layers keep their keys
                                whole (K pools of width D, nothing of K is predicted, Wk may be NULL) and only the
                                values are evicted and predicted.  Decode calls are served by the absorbed mode
                                only (EUNSUPPORTED until echokv_enable_absorbed) */
} echokv_config;

typedef struct {
  uint64_t anchor_pool_bytes;     /* one K (or V) pool of an anchor layer                  */
  uint64_t compressed_pool_bytes; /* one K (or V) pool of a compressed layer (0 if m = 0); with
                                     save_k the K pools of compressed layers have anchor_pool_bytes */
  uint64_t block_table_bytes;
  uint64_t workspace_bytes;       /* minimum size of echokv_buffers.workspace              */
  int32_t max_partials;           /* split-K partial results kept per (sequence, head)     */
  int32_t reserved;
} echokv_sizes;

typedef struct {
  void* const* k_pools;      /* host array [n_layers] of device pointers (copied at create) */
  void* const* v_pools;      /* same for V; entries of compressed layers may be NULL if m=0 */
  void* workspace;           /* device pointer, >= workspace_bytes, 256-byte aligned        */
  uint64_t workspace_bytes;
} echokv_buffers;

/* Sizes implied by a config.  Pure host arithmetic, no CUDA call.
 * Errors: EINVAL (NULL or inconsistent config), EUNSUPPORTED (head_dim, page size). */
int echokv_query_sizes(const echokv_config* cfg, echokv_sizes* out);

/* Build a context over caller-owned device buffers (pools, workspace).  Makes `device`
 * current, clears the workspace's status word (synchronous) and prepares the tensor maps
 * of every pool.  Errors: EINVAL, EUNSUPPORTED, ECAPACITY (workspace too small), ECUDA. */
int echokv_create(const echokv_config* cfg, const echokv_buffers* buffers, echokv_ctx** out);

/* Release the context (host memory only; the caller's device buffers are untouched). */
void echokv_destroy(echokv_ctx* ctx);

/* Install the predictors of compressed layer `layer` (Eq. 3): device pointers Wk, Wv of
 * [D - m][D + m] elements, optional biases bk, bv of [D - m] (NULL = none, the paper's
 * Eq. 3 has none).  Borrowed.  Errors: EINVAL, ENOTCOMPRESSED, ECUDA. */
int echokv_set_weights(echokv_ctx* ctx, int layer, const void* Wk, const void* Wv,
                       const void* bk, const void* bv);

/* Install the block table: device pointer to int32 [max_batch][max_pages_per_seq].
 * Borrowed; the caller may change its contents between calls (stream-ordered). */
int echokv_set_block_table(echokv_ctx* ctx, const int32_t* dev_block_table);

/* Append one new token per sequence to layer `layer`'s cache (Section 3.1: compression is
 * plain eviction of part of each token's K/V): k_new, v_new are device pointers
 * [B][n_kv_heads][head_dim];
 * an anchor layer stores all D dims, a compressed layer only the first m (Eq. 2) -- the rest
 * is never written anywhere.  dev_positions[b] = token index to write (its page must be in
 * the block table); dev_seq_slots[b] = row of the block table (NULL = row b).
 * Bad slot / page / position -> device status EBADPAGE, that token is skipped.
 * Errors: EINVAL, ECAPACITY, ENOTABLE, ECUDA. */
int echokv_append_kv(echokv_ctx* ctx, int layer, const void* k_new, const void* v_new,
                     const int32_t* dev_seq_slots, const int32_t* dev_positions, int B, void* stream);

/* The same for n_tokens consecutive new tokens per sequence (a chunk of a prompt during prefill): k_new, v_new are
 * device pointers [B][n_tokens][n_kv_heads][head_dim], dev_first_positions[b] = position of the first of them.  With
 * a sink / window set, of the chunk's tokens only the last n_window enter the window ring (the others would be
 * overwritten by them anyway).  echokv_append_kv is this call with n_tokens = 1.
 * Errors: as echokv_append_kv; ECAPACITY also if n_tokens exceeds 65535 or the sequence capacity. */
int echokv_append_kv_chunk(echokv_ctx* ctx, int layer, const void* k_new, const void* v_new,
                           const int32_t* dev_seq_slots, const int32_t* dev_first_positions, int n_tokens, int B,
                           void* stream);

/* The switch from full-cache generation to compressed inference (Section 3.1: compression is evicting part
 * of each token's K / V, at the moment memory runs short; Section 5.4: or already during prefill).  The caller
 * has cached layer `layer` at full width in pools of its own, k_full / v_full: device pointers
 * [n_pages][page_tokens][D] (16-byte aligned) addressed by the same block table.  For tokens
 * dev_seq_begins[b] .. dev_seq_lens[b]-1 of each of the B sequences the call copies dims 0 .. m-1 of K and V
 * into the layer's own pools (Eq. 2) and, while a sink / window is set, dims m .. D-1 of the sink tokens and of
 * the last n_window tokens before dev_seq_lens[b] into the side buffers; afterwards echokv_decode_attention
 * serves the layer and the caller may release the full-width pools.  With save_k the keys are copied whole and the
 * side buffers receive values only.  dev_seq_begins = NULL means 0; with a
 * prefill done in chunks, call it once per chunk with the chunk's range.  The copies are bit-exact.
 * Bad slot / page -> device status EBADPAGE, bad length or begin -> EBADLENGTH; that sequence is skipped.
 * Errors: EINVAL, ENOTCOMPRESSED (anchor layers keep everything), ECAPACITY, ENOTABLE, ECUDA. */
int echokv_compress_layer(echokv_ctx* ctx, int layer, const void* k_full, const void* v_full,
                          const int32_t* dev_seq_slots, const int32_t* dev_seq_begins,
                          const int32_t* dev_seq_lens, int B, void* stream);

/* Decode attention of compressed layer `layer` (Eq. 3, 6, 7): q is a device pointer
 * [B][n_q_heads][head_dim], out a device pointer to fp32 [B][n_q_heads][head_dim],
 * dev_seq_lens[b] = tokens in the cache (>= 1, newest included).  Heads 0..r-1 attend their
 * stored K/V; heads r.. attend K/V predicted on chip from the anchor layer's cache and this
 * layer's retained dims.  Called on an anchor layer it is the same as echokv_full_attention.
 * Uses the workspace; calls on one context must not overlap on the device.
 * A length < 1 or beyond max_pages_per_seq * page_tokens -> device status EBADLENGTH and
 * zeros for that sequence.  A page id outside the pool (a caller's error) -> device status EBADPAGE; nothing is
 * read through it and every other sequence of the call is unaffected, but the output of the sequence it belongs
 * to is unspecified: the stored-head kernels leave the page's tokens out, the tensor-core kernels find whatever
 * rows their staging memory held in their place.
 * Errors: EINVAL, ECAPACITY, ENOWEIGHTS, ENOTABLE, ECUDA. */
int echokv_decode_attention(echokv_ctx* ctx, int layer, const void* q, float* out,
                            const int32_t* dev_seq_slots, const int32_t* dev_seq_lens, int B,
                            void* stream);

/* Prefill-shaped attention: the last n_q cached tokens of every sequence are queries at once (a later chunk of
 * a prompt whose earlier chunks were already evicted down to the compressed cache: Section 5.4, "drop unnecessary
 * cache entries during the pre-filling phase").  Query i of sequence b sits at position dev_seq_lens[b] - n_q + i
 * and attends the tokens up to and including its own (causal); its own K / V must already be in the cache.
 * q: device pointer [B][n_q][n_q_heads][head_dim]; out: device pointer to fp32 of the same shape.
 * With many queries the cache is rebuilt once per call rather than once per query: the stored dims are gathered
 * and the dropped dims predicted (Eq. 3, on the tensor cores; K bias and rotary table applied if set) into
 * `scratch`, a caller-owned device buffer of echokv_prefill_scratch_bytes() bytes (16-byte aligned) that holds K~
 * and V~ as bf16 rows [B][max_pages_per_seq * page_tokens][D] each (plus one float per sequence, query and query
 * head), and a causal attention kernel runs over those rows.  Unlike the decode calls this one does round the
 * predicted K and V to bf16 (as the paper's own materialise-then-attend implementation does).  Works on anchor
 * layers too (nothing is predicted there).  bf16, head_dim 128 only (EUNSUPPORTED otherwise); m may split a head.
 * With save_k the keys are gathered whole and only the values are predicted.
 * With sink / window tokens set (Section 4.1) every query is the decode step of the sequence cut off at its own
 * position: it reads the first n_sink tokens and ITS OWN last n_window tokens at full precision and every other
 * token as predicted.  The side buffers hold the window of the end of the sequence only, so the call then takes the
 * recent tokens' rows from the caller: k_recent, v_recent are device pointers (16-byte aligned, EINVAL if NULL) to
 * [B][n_q + n_window - 1][n_kv_heads][head_dim], the whole K and V rows of positions dev_seq_lens[b] - n_q -
 * n_window + 1 .. dev_seq_lens[b] - 1 -- the chunk itself preceded by the n_window - 1 tokens before it; rows of
 * positions below 0 are not read.  Without a window (and on anchor layers) both are ignored and may be NULL.
 * A sequence with fewer than n_q cached tokens, or an unusable slot / length: zeros and the device status.
 * Errors: EINVAL, EUNSUPPORTED, ECAPACITY (batch, scratch too small), ENOWEIGHTS, ENOTABLE, ECUDA. */
int echokv_prefill_scratch_bytes(const echokv_config* cfg, uint64_t* out);
int echokv_prefill_attention(echokv_ctx* ctx, int layer, const void* q, float* out, int n_q,
                             const int32_t* dev_seq_slots, const int32_t* dev_seq_lens, int B,
                             const void* k_recent, const void* v_recent,
                             void* scratch, uint64_t scratch_bytes, void* stream);

/* Attention over a layer that holds its full cache (anchor layers; the uncompressed
 * short-context mode the paper switches from, Section 5.4): Eq. 7 on the stored K, V.
 * Same arguments as echokv_decode_attention.  Errors: as above plus ENOTANCHOR. */
int echokv_full_attention(echokv_ctx* ctx, int layer, const void* q, float* out,
                          const int32_t* dev_seq_slots, const int32_t* dev_seq_lens, int B,
                          void* stream);

/* One layer-step driven from HOST memory: copies q, k_new, v_new ([B][heads][head_dim],
 * storage dtype) and seq_lens (int32 [B], lengths AFTER the append) to the device, appends
 * at position seq_lens[b]-1 in block-table row b, runs the layer's attention if `attend`
 * is non-zero (decode for a compressed layer, full for an anchor), copies the fp32 result to
 * out_host and synchronises the stream.  For best speed the host buffers should be pinned.
 * q_host / out_host may be NULL when attend == 0.  Errors: as the calls it is made of. */
int echokv_layer_step_host(echokv_ctx* ctx, int layer, const void* q_host, const void* k_new_host,
                           const void* v_new_host, float* out_host, const int32_t* seq_lens_host,
                           int B, int attend, void* stream);

/* Read and clear the device status word (synchronises the device).  *host_out receives
 * ECHOKV_OK or the first device-side error (ETIMEOUT, EBADPAGE, EBADLENGTH). */
int echokv_get_device_status(echokv_ctx* ctx, int32_t* host_out);

/* Sink and recent-window tokens at full precision (Section 4.1, "Implement details": the paper keeps
 * 4 sink tokens and a local window of 128 tokens uncompressed).  With (n_sink, n_window) set, the first
 * n_sink and the last n_window tokens of every sequence are never predicted: the dims m .. D-1 of those
 * tokens are kept in per-layer side buffers and Eq. 7 uses them as stored; every other token is
 * reconstructed by Eq. 3 as before.
 *  - echokv_side_buffer_bytes: size of ONE side buffer: [max_batch][n_sink + n_window][D - m] elements
 *    of the storage dtype.  EUNSUPPORTED if n_sink + n_window > 4096.
 *  - echokv_set_full_precision_window: k_side / v_side are host arrays [n_layers] of device pointers
 *    (16-byte aligned, borrowed; entries of anchor layers are ignored and may be NULL; with save_k the keys
 *    are whole in the pools already and k_side itself may be NULL).  From then on
 *    echokv_append_kv on a compressed layer also writes the new token's dims m .. D-1 to the side buffers
 *    (slot `position` while position < n_sink, and ring slot n_sink + position % n_window), and
 *    echokv_decode_attention attends the sink / window tokens from there.  Set it before the first
 *    append, or fill the slots of the tokens already cached yourself.  (0, 0) switches it off.
 *    Works in both decode modes.  Errors: EINVAL, EUNSUPPORTED. */
int echokv_side_buffer_bytes(const echokv_config* cfg, int n_sink, int n_window, uint64_t* out);
int echokv_set_full_precision_window(echokv_ctx* ctx, int n_sink, int n_window, void* const* k_side,
                                     void* const* v_side);

/* Rotary position embedding applied when the cache is read.  Section 3.2 feeds the predictors keys PRIOR
 * to RoPE, so a backbone that follows the paper caches un-rotated keys and the rotation has to happen between
 * reconstruction and q . k.  With a rotary table set, every attention call of the context rotates row t of
 * K~ (stored, predicted, sink / window alike; anchor layers and echokv_full_attention included) to position
 * t before the dot product:  feature j < head_dim/2 pairs with feature j + head_dim/2 (the Llama layout),
 *     k'[j] = k[j] cos(a) - k[j + d/2] sin(a),  k'[j + d/2] = k[j + d/2] cos(a) + k[j] sin(a),
 *     a = t * theta^(-2 j / head_dim),  t = index of the token in its sequence.
 * q must arrive already rotated to its own position; V is never rotated.  The paper does not say where the
 * rotation is re-applied at inference; this is the reading that keeps Eq. 3 on un-rotated keys.
 *  - echokv_rope_table_bytes: size of the table, [head_dim / 2][max_pages_per_seq * page_tokens] pairs
 *    (cos, sin) of fp32.
 *  - echokv_set_rope: `table` is a device pointer of at least that size (16-byte aligned, borrowed until
 *    echokv_destroy or until rope is switched off); the call enqueues one kernel on `stream` that fills it
 *    (angles and sin / cos in fp64, rounded to fp32 once) and switches rotation on for later calls.
 *    theta = 0 with table = NULL switches it off.  In the absorbed mode a rotation that depends on the token cannot be folded into the
 *    queries: with a table set that mode evaluates the K side explicitly (predicted keys on the tensor cores,
 *    rotated, scored) and keeps the absorbed form for the V side only -- about half the tensor work of the
 *    explicit mode.  Errors: EINVAL (theta < 1, misaligned), ECAPACITY, EUNSUPPORTED, ECUDA. */
int echokv_rope_table_bytes(const echokv_config* cfg, uint64_t* out);
int echokv_set_rope(echokv_ctx* ctx, double theta, void* table, uint64_t table_bytes, void* stream);
int echokv_rope_enabled(const echokv_ctx* ctx);

/* Absorbed-predictor decode mode.  Eq. 3 is linear, so Eq. 7 over a predicted head can be evaluated
 * without forming the predicted K and V:
 *     q . (Wk x_t) = (Wk^T q) . x_t          sum_t p_t (Wv x_t) = Wv (sum_t p_t x_t)
 * with x_t = [anchor dims ; retained dims] of token t.  The library then streams the K features once
 * (scores of all query heads against "absorbed queries" Wk^T q), the V features once (probability-
 * weighted sums of x_t) and applies Wv at the end: the same function of the same inputs as
 * echokv_decode_attention's default (explicit) mode up to rounding, at about D_drop / (2 n_q_heads)
 * times fewer FLOPs, bound by HBM bandwidth instead of the tensor cores.  The paper does not describe
 * this evaluation order; it follows from the linearity of its predictor (Section 3.2, Eq. 3).
 *
 *  - echokv_absorbed_workspace_bytes: size of the extra device workspace the mode needs (scores and
 *    probabilities of every cached token and head, absorbed queries, partial sums).
 *    EUNSUPPORTED unless dtype is bf16, head_dim 128, n_q_heads in {16, 32, 64}, at least one head is
 *    dropped and max_batch <= 256.
 *  - echokv_enable_absorbed: hands the library that workspace (device pointer, 256-byte aligned,
 *    borrowed until echokv_destroy) and switches the context to the absorbed mode.
 *    Errors: EINVAL, EUNSUPPORTED, ECAPACITY (workspace too small), ECUDA.
 *  - echokv_set_decode_mode: 0 = explicit reconstruction, 1 = absorbed (EUNSUPPORTED before
 *    echokv_enable_absorbed).  Anchor layers and echokv_full_attention are not affected.
 *  A page id outside the pool: as for echokv_decode_attention. */
int echokv_absorbed_workspace_bytes(const echokv_config* cfg, uint64_t* out);
int echokv_enable_absorbed(echokv_ctx* ctx, void* workspace, uint64_t workspace_bytes);
int echokv_decode_mode(const echokv_ctx* ctx);
int echokv_set_decode_mode(echokv_ctx* ctx, int mode);

/* Full-cache attention for callers that cannot allocate device memory (the paper has no
 * counterpart to this entry point; it exists for the library's users).
 *
 * Every other attention call needs a context whose split-K workspace the caller allocated.  A
 * caller that is only ever handed raw pointers -- a plug-in running inside another framework's
 * execution callback where allocation is forbidden, a thread that works out of an arena sized
 * long ago -- has no way to provide one.  This call needs no context and no workspace: it
 * computes what echokv_full_attention computes (Eq. 7 on the stored cache of one layer), taking
 * the layer's pools, the block table, q, out and the lengths directly, and keeps its partial
 * results in a fixed array inside the library image: echokv_noalloc_scratch_bytes() bytes
 * (8 MiB), resident on every GPU that loads the library until the process exits.
 *
 *  - cfg describes the geometry (heads, head_dim, page_tokens, max_batch, max_pages_per_seq,
 *    n_pages, dtype, softmax_scale, device); n_layers, group_size, n_retained_heads are ignored.
 *    k_pool / v_pool: device pointers [n_pages][page_tokens][n_kv_heads * head_dim]; the other
 *    pointers as in echokv_full_attention (k_pool, v_pool, q and out 16-byte aligned, else EINVAL;
 *    max_pages_per_seq * page_tokens at most 2^30).  dev_status_out: optional device int32 that receives
 *    the device status of this call (ECHOKV_OK, EBADPAGE, EBADLENGTH), stream-ordered.
 *  - It calls no cudaMalloc / cudaFree and no routine that allocates.  Makes cfg->device current.
 *  - The FIRST call on each device looks up the device address of the array; make that first
 *    call before any stream capture begins.
 *  - Size limit: B * n_q_heads * (8 + 4 * head_dim) + 256 bytes must fit the array (for
 *    head_dim 128: B * n_q_heads <= 16131); beyond it the call returns ECHOKV_ESCRATCH and does
 *    nothing.  Fewer sequence splits are used when more would not fit.
 *  - All calls, on all streams and from all threads, share the one array per device, and it keeps
 *    whatever the previous call left in it (the call clears the one word it needs cleared).
 *    Two calls that overlap on the GPU race on it: order them, e.g. on one stream.
 * Errors: EINVAL, EUNSUPPORTED, ECAPACITY (B > max_batch), ESCRATCH, ECUDA. */
int echokv_full_attention_noalloc(const echokv_config* cfg, const void* k_pool, const void* v_pool,
                                  const int32_t* dev_block_table, const void* q, float* out,
                                  const int32_t* dev_seq_slots, const int32_t* dev_seq_lens, int B,
                                  int32_t* dev_status_out, void* stream);

/* Size in bytes of the fixed scratch array behind echokv_full_attention_noalloc. */
uint64_t echokv_noalloc_scratch_bytes(void);

/* =====================================================================================================
 * Diagnostics: switches, counters and probes for tests and benchmarks.  No product call depends on them;
 * contexts start on the fastest kernels their shape allows.
 * ===================================================================================================== */

/* Number of kernels the library has launched on this context since creation. */
int64_t echokv_launch_count(const echokv_ctx* ctx);

/* Which kernel family serves compressed layers of this context:
 * 0 = none (no layer is compressed or nothing is dropped), 1 = fp32/bf16 CUDA-core kernel,
 * 2 = bf16 tcgen05 tensor-core kernel, one CTA per SM, 3 = the same on CTA pairs
 * (cta_group::2: two SMs share every operand tile and the accumulators are double-buffered),
 * 4 = CTA pairs with four dropped heads per work item (a token tile staged once per four heads),
 * 5 = 2 or 4, decided on the device at every call by the page order found in the block table (pages handed out in
 *     order: 2, which fetches four consecutive pages as one copy; otherwise 4, which is indifferent to the order). */
int echokv_decode_path(const echokv_ctx* ctx);

/* After a decode call on path 5 (synchronises the device): *out = 1 if that call found the pages in order (kernel
 * family 2 ran), 0 if not (family 4 ran).  EINVAL on another path. */
int echokv_diag_page_order(echokv_ctx* ctx, int32_t* out);

/* Choose the kernel family for compressed layers: 1 = CUDA-core kernel (always possible),
 * 2, 3, 4 or 5 = tcgen05 kernels (EUNSUPPORTED unless dtype is bf16, head_dim 128; 4 and 5 also need at most two
 * query heads per KV head, 5 pages of at most 32 tokens).  Contexts start on the fastest family their shape allows.  Meant for tests that check all
 * against the oracle. */
int echokv_set_decode_path(echokv_ctx* ctx, int path);

/* Which kernel serves attention over stored heads (anchor layers, retained heads, the
 * uncompressed mode): 0 = CUDA-core kernel (any supported shape), 1 = TMA + tensor-core kernel
 * (bf16, head_dim 128).  Contexts start on 1 when their shape allows it.
 * echokv_set_stored_path: EINVAL (not 0 or 1), EUNSUPPORTED (1 on a shape it does not take).
 * Meant for tests that check both against the oracle. */
int echokv_stored_path(const echokv_ctx* ctx);
int echokv_set_stored_path(echokv_ctx* ctx, int path);

/* Device timing of the dominant kernel of each attention call (the fused reconstruct-attend
 * kernel on compressed layers, the stored-head attention kernel on anchor layers): when enabled,
 * the library records a CUDA event pair around that kernel on the call's stream.
 * echokv_read_kernel_timing synchronises the device, returns the summed duration and the number
 * of timed launches since the last read, and starts over.  Errors: EINVAL, ECUDA. */
int echokv_set_kernel_timing(echokv_ctx* ctx, int enable);
int echokv_read_kernel_timing(echokv_ctx* ctx, double* total_ms, int64_t* n_launches);

/* The same reading split by kernel: total_ms and n_launches are host arrays of
 * ECHOKV_TIMED_KINDS entries, indexed by ECHOKV_TIMED_STORED (stored-head attention of an
 * anchor / uncompressed layer), ECHOKV_TIMED_RECON (fused reconstruct-attend kernel) and the two
 * streaming kernels of the absorbed mode. */
enum {
  ECHOKV_TIMED_STORED = 0, ECHOKV_TIMED_RECON = 1,
  ECHOKV_TIMED_ABSORB_K = 2,   /* absorbed mode: the pass over the K features (scores)          */
  ECHOKV_TIMED_ABSORB_V = 3,   /* absorbed mode: the pass over the V features (weighted sums)   */
  ECHOKV_TIMED_KINDS = 4
};
int echokv_read_kernel_timing_by_kind(echokv_ctx* ctx, double* total_ms, int64_t* n_launches);

/* The give-up path of the kernels' bounded waits, exercised without a fault: enqueues one small block that waits,
 * with the same routine the kernels use and a limit of limit_cycles SM cycles (1 .. 2e9), on a barrier nothing ever
 * arrives on.  The waiting warp raises ECHOKV_ETIMEOUT in the device status word (read it with
 * echokv_get_device_status) and a flag that releases the block's other waiting warp, as a kernel's other roles are
 * released; the block issues no copy and allocates no tensor memory, so nothing is pending when it returns and the
 * context stays usable.  dev_left_by: device pointer to int32[2], how each of the two warps left (1 = gave up or was
 * released by the flag, 0 = its barrier completed, which cannot happen).  Errors: EINVAL, ECUDA. */
int echokv_diag_bounded_wait(echokv_ctx* ctx, int64_t limit_cycles, int32_t* dev_left_by, void* stream);

/* Static, human-readable name of a status code. */
const char* echokv_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ECHOKV_H */
