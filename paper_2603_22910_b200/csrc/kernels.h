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
};

// Append one token per sequence: writes the first `width` flat dims of k_new / v_new.
cudaError_t launch_append(int dtype, void* k_pool, void* v_pool, int width, int D, const void* k_new,
                          const void* v_new, const int32_t* slots, const int32_t* positions, int B,
                          const PageGeom& geom, int32_t* status, cudaStream_t stream);

// Attention of query heads whose KV head is stored (heads 0..n_heads-1 of a pool of row width
// `width`), split over the sequence into n_splits partials per head.
cudaError_t launch_attn_stored(const AttnArgs& a, const void* k_pool, const void* v_pool, int width,
                               int n_heads, int n_splits, cudaStream_t stream);

struct ReconArgs {
  const void* k_anchor; const void* v_anchor;   // pools of row width D
  const void* k_local; const void* v_local;     // pools of row width m (may be null when m == 0)
  const void* Wk; const void* Wv;               // [D - m][D + m]
  int D, m;
  int part_tokens;                              // tokens per partial
  int capacity_tokens;                          // max_pages_per_seq * page_tokens
};

// CUDA-core reconstruct-then-attend (fp32 or bf16 storage, fp32 FFMA): Eq. 3, 6, 7 for the
// dropped KV heads; one partial per part_tokens tokens.
cudaError_t launch_recon_simt(const AttnArgs& a, const ReconArgs& r, cudaStream_t stream);

// Merge split-K partials into out[B][H_q][d].  Heads with KV head < n_stored_heads have
// n_stored_parts partials or, when stored_item_tokens is given (device; one entry per
// stored_batch_per_slot sequences, written by the stored-head kernel), ceil(len / that entry);
// the others ceil(len / part_tokens).  bv (may be null): bias of the V predictor, fp32-converted
// on the fly, added to dropped heads ([D - m] in storage dtype).
cudaError_t launch_merge(const AttnArgs& a, float* out, int n_stored_heads, int n_stored_parts,
                         const int32_t* stored_item_tokens, int stored_batch_per_slot, int part_tokens,
                         const void* bv, cudaStream_t stream);

}  // namespace echokv
