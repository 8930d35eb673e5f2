// Host-side launchers of the EchoKV kernels (internal to the library).
#pragma once

#include "common.cuh"

namespace echokv {

struct AttnArgs {
  int dtype;                 // ECHOKV_BF16 / ECHOKV_FP32
  int n_q_heads, n_kv_heads, head_dim;
  int batch;
  float scale_log2e;         // softmax scale * log2(e)
  const void* q;             // [B][H_q][d]
  const int32_t* slots;      // [B] or null
  const int32_t* lens;       // [B]
  PageGeom geom;
  Partials parts;
  int32_t* status;
  RopeTable rope;            // rotate every key row to its position before q . k (off unless set)
};

// The three parts of a rotary table (see RopeTable) live in one buffer: [d/2][stride], then [stride/16][d/2],
// then [16][d/2] pairs.  rope_table_pairs: pairs in all; rope_table_view: the RopeTable over such a buffer;
// launch_rope_table: fill it (angles and sin / cos in fp64; three launches).
size_t rope_table_pairs(int stride, int head_dim);
RopeTable rope_table_view(const float2* buffer, int stride, int head_dim);
cudaError_t launch_rope_table(float2* buffer, int stride, int head_dim, double theta, cudaStream_t stream);

// Append n_tokens consecutive tokens per sequence (k_new / v_new: [B][n_tokens][D]; positions[b] = where the first
// one goes): writes the first k_width flat dims of every new K row and the first v_width of every new V row.
cudaError_t launch_append(int dtype, void* k_pool, void* v_pool, int k_width, int v_width, int D, const void* k_new,
                          const void* v_new, const int32_t* slots, const int32_t* positions, int B, int n_tokens,
                          const PageGeom& geom, int32_t* status, cudaStream_t stream);

// Attention of query heads whose KV head is stored (heads 0..n_heads-1 of a pool of row width
// `width`), split over the sequence into n_splits partials per head.
cudaError_t launch_attn_stored(const AttnArgs& a, const void* k_pool, const void* v_pool, int width,
                               int n_heads, int n_splits, cudaStream_t stream);

struct ReconArgs {
  const void* k_anchor; const void* v_anchor;   // pools of row width D
  const void* k_local; const void* v_local;     // pools of row width m (may be null when m == 0)
  const void* Wk; const void* Wv;               // [D - m][D + m]
  const void* bk = nullptr;                     // bias of the K predictor [D - m], or null.  Only read when the keys
                                                // are rotated after prediction: without a rotation it shifts every
                                                // score of a head alike and cancels in the softmax
  int D, m;
  int m_heads = -1;                             // flat dims of the WHOLE retained heads (a multiple of head_dim, <= m);
                                                // -1: m.  Where m splits a head, the split head counts as predicted:
                                                // Wk, Wv, bk then have D - m_heads rows, the first m - m_heads of
                                                // them passing the head's stored dims through (one-hot rows)
  int part_tokens;                              // tokens per partial
  int capacity_tokens;                          // max_pages_per_seq * page_tokens
  int n_sink = 0, n_window = 0;                 // tokens kept at full precision: the first n_sink and the last
                                                // n_window of a sequence are NOT predicted here (they are
                                                // attended from the side buffers, see launch_attn_side)
  // Two kernels launched for the same work, one of which does it: a kernel given `choose` runs only if the device
  // word holds choose_value (see launch_page_order), else it returns at once.  Null: run.
  const int32_t* choose = nullptr;
  int choose_value = 0;
};

// *flag (device) = 1 if most of the sequences' aligned 64-token groups lie on consecutive pool rows (their pages were
// handed out in order), else 0: the one-CTA fused kernel fetches such a group as one copy and is the faster one
// there, the four-head CTA-pair kernel is indifferent to the page order (a sample of the groups is looked at).
cudaError_t launch_page_order(const AttnArgs& a, int32_t* flag, cudaStream_t stream);

// Whole retained heads of a compressed layer (the kernels' first predicted head).
__host__ __device__ inline int retained_heads(const ReconArgs& r, int head_dim) { return (r.m_heads >= 0 ? r.m_heads : r.m) / head_dim; }

// Predictor [d_drop][d_in] (+ bias [d_drop] or null) -> Wx [split + d_drop][d_in] (+ bx, may be null): `split`
// one-hot rows in front that pass input columns pass_col0 .. pass_col0 + split - 1 through unchanged.
cudaError_t launch_extend_predictor(int dtype, const void* W, const void* bias, void* Wx, void* bx, int d_drop,
                                    int d_in, int split, int pass_col0, cudaStream_t stream);

// Tokens of a sequence of `len` tokens that are predicted: [lo, hi) (Section 4.1: sink and recent-window
// tokens keep all their dims).
__host__ __device__ inline int predicted_lo(int len, int n_sink) { return n_sink < len ? n_sink : len; }
__host__ __device__ inline int predicted_hi(int len, int n_sink, int n_window) {
  const int lo = predicted_lo(len, n_sink);
  const int hi = len - n_window;
  return hi > lo ? hi : lo;
}

// Side buffers of one compressed layer: the dropped dims (m .. D-1) of the sink and recent-window tokens,
// [max_batch][n_sink + n_window][D - m] in the storage dtype; slot of token t: t if t < n_sink, and
// n_sink + t % n_window while it is inside the window.
struct SideArgs {
  void* k_side; void* v_side;
  int n_sink, n_window, d_drop;
};

// Append: the new tokens' dropped dims go to their side slots.
cudaError_t launch_append_side(int dtype, const SideArgs& side, int m, int D, const void* k_new, const void* v_new,
                               const int32_t* slots, const int32_t* positions, int B, int n_tokens, int max_batch,
                               int32_t* status, cudaStream_t stream);

// Evict a full-width cache ([n_pages][page_tokens][D], same block table) down to what a compressed layer keeps:
// dims 0 .. mk-1 of the keys and 0 .. m-1 of the values of tokens [begins[b], lens[b]) into k_local / v_local
// (skipped when 0), dims m .. D-1 of the sink / window tokens (window relative to lens[b]) into the side buffers
// (side may be null; side->k_side may be null: keys kept whole).  Bit-exact copies.
cudaError_t launch_compress(int elem_bytes, const void* k_full, const void* v_full, void* k_local, void* v_local,
                            const SideArgs* side, int D, int mk, int m, const int32_t* slots, const int32_t* begins,
                            const int32_t* lens, int B, const PageGeom& geom, int32_t* status, cudaStream_t stream);

// Eq. 7 over the sink and window tokens, at full precision, for the KV heads first_head .. n_kv_heads-1: one
// split-K partial per (sequence, query head), written at partial index pool.part, or ceil(len / part_tokens)
// when that is < 0.  Of every head the dims below pool.width (= m) come from the layer's pools and the rest from
// the side buffers, so the call serves dropped heads, a head that m splits, and (the absorbed mode, first_head = 0)
// retained heads alike.
struct SidePool {
  const void* k_pool; const void* v_pool;   // the layer's pools (row width `width` = m; may be null when m == 0)
  int width;
  int part;
  int k_width = 0;                          // row width of the K pool where it differs (keys kept whole: D); 0: width
};
// choose / alt_part_tokens: where two fused kernels with different partial sizes were launched for the same work
// (ReconArgs::choose), the partials are alt_part_tokens long if *choose == 1, else part_tokens.
cudaError_t launch_attn_side(const AttnArgs& a, const SideArgs& side, int first_head, int part_tokens,
                             cudaStream_t stream, const SidePool& pool, const int32_t* choose = nullptr,
                             int alt_part_tokens = 0);

// CUDA-core reconstruct-then-attend (fp32 or bf16 storage, fp32 FFMA): Eq. 3, 6, 7 for the
// dropped KV heads; one partial per part_tokens tokens.
cudaError_t launch_recon_simt(const AttnArgs& a, const ReconArgs& r, cudaStream_t stream);

// Merge split-K partials into out[B][H_q][d].  Heads with KV head < n_stored_heads have
// n_stored_parts partials or, when stored_item_tokens is given (device; one entry per
// stored_batch_per_slot sequences, written by the stored-head kernel), ceil(len / that entry);
// the others ceil(len / part_tokens).  bv (may be null): bias of the V predictor, fp32-converted
// on the fly, added to dropped heads ([D - m] in storage dtype) with the predicted tokens' share of the probability.
// extra_recon_part = 1: the dropped heads have one more partial, their last, over the sink / window tokens.
// bk_shift (may be null): bias of the K predictor where the kernels left it out of the scores; it then moves the
// predicted partials of a head by q . b_k against that sink / window partial (without one it cancels).
cudaError_t launch_merge(const AttnArgs& a, float* out, int n_stored_heads, int n_stored_parts,
                         const int32_t* stored_item_tokens, int stored_batch_per_slot, int part_tokens,
                         const void* bv, cudaStream_t stream, int extra_recon_part = 0,
                         const void* bk_shift = nullptr, const int32_t* choose = nullptr, int alt_part_tokens = 0);

}  // namespace echokv
