// Tensor-core (mma.sync) + TMA attention over stored bf16 heads of 128 dims: host interface.
#pragma once

#include <cuda.h>

#include "kernels.h"

namespace echokv {

constexpr int kStoredMaxBatchPerLaunch = 512;   // sequences one launch indexes in shared memory
constexpr int kStoredMaxLaunches = 32;          // launches (and published item sizes) per call

bool stored_mma_supported(int dtype, int head_dim, int group, int max_batch);

// Token rows per TMA box of the pool maps this kernel wants: min(page_tokens, 64); 64 features wide.
int stored_rows_per_box(int page_tokens);

// Eq. 7 for the query heads of KV heads 0 .. n_heads-1 of the pool behind k_map / v_map.  One
// split-K partial per (sequence, item, query head), item = a range of item_tokens tokens; the
// kernel chooses item_tokens and writes it to item_tokens_slots[launch index] (one launch per
// kStoredMaxBatchPerLaunch sequences) for the merge kernel.
// k_run_map / v_run_map: the same pools in boxes of 64 token rows (used when a stage's pages are consecutive).
cudaError_t launch_attn_stored_mma(const AttnArgs& a, const CUtensorMap& k_map, const CUtensorMap& v_map,
                                   const CUtensorMap& k_run_map, const CUtensorMap& v_run_map, int n_heads, int32_t* item_tokens_slots, int sm_count, cudaStream_t stream);

// Scores of stored heads whose keys are rotated when read: S[b][h][t] = q_h . R_t k_t (base-2 units) for the query
// heads of KV heads 0 .. n_heads-1 of the pool behind k_map / k_run_map; token slots of a sequence's whole 256-token
// tiles that hold no predicted token get -inf.  Feeds the softmax of the absorbed V side when the K side has to be
// explicit (rotated keys).  S: [batch][n_q_heads][l_cap].
cudaError_t launch_key_scores_stored(const AttnArgs& a, const CUtensorMap& k_map, const CUtensorMap& k_run_map,
                                     int n_heads, float* S, int l_cap, int n_sink, int n_window, int sm_count,
                                     cudaStream_t stream);

}  // namespace echokv
