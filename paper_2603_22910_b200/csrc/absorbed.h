// Absorbed-predictor decode: host interface.
//
// Eq. 3 is linear, so Eq. 7 over predicted heads can be evaluated without ever forming the
// predicted K and V:  q . (W_k x_t) = (W_k^T q) . x_t   and   sum_t p_t (W_v x_t) = W_v (sum_t p_t x_t).
// Every query head then attends over the same per-token vector x_t = [anchor dims ; retained dims]
// (a retained head's "absorbed query" simply selects its own dims), which makes the layer one
// stream over the K features, one stream over the V features and two small projections.
#pragma once

#include <cuda.h>

#include "recon_tc.h"

namespace echokv {

constexpr int kAbsorbMaxRanges = 16;     // token ranges the V pass may split a sequence into
constexpr int kAbsorbTokAlign = 128;     // score rows are padded to this many tokens

struct AbsorbLayout {
  int nh2;          // rows of the absorbed-query / probability matrices per sequence: 2 * n_q_heads (hi, lo)
  int l_cap;        // tokens per score row
  uint64_t off_q2;  // bf16 [max_batch * nh2][D_in]      absorbed queries, split into two bf16 halves
  uint64_t off_s;   // fp32 [max_batch][n_q_heads][l_cap] scores (base-2 units)
  uint64_t off_p2;  // bf16 [max_batch * nh2][l_cap]     probabilities, split into two bf16 halves
  uint64_t off_ml;  // float2 [max_batch][n_q_heads]      (max, sum) of every head
  uint64_t off_ml_range;  // float2 [max_batch][n_q_heads][ranges]  the same per token range
  uint64_t off_y;   // fp32 [max_batch][ranges][n_q_heads][D_in]  partial probability-weighted inputs
  uint64_t off_ysum; // fp32 [max_batch][n_q_heads][D_in]         their sum over ranges, divided by the softmax sum
  uint64_t total;
};

// m = retained flat dims per token: any multiple of 64 below D (it need not end on a head boundary)
bool absorbed_supported(int dtype, int head_dim, int n_q_heads, int n_kv_heads, int m, int page_tokens);
void absorbed_layout(int max_batch, int n_q_heads, int d_in, int capacity_tokens, AbsorbLayout* out);

struct AbsorbMaps {
  CUtensorMap q2;   // [chunk][row][64] view of the absorbed queries, boxes of 2 chunks x nh2 rows
  CUtensorMap p2;   // probabilities, boxes of nh2 rows x 64 tokens
  bool ready = false;
};

cudaError_t absorbed_encode_maps(AbsorbMaps* maps, unsigned char* ws, const AbsorbLayout& lay, int max_batch, int d_in);

struct AbsorbArgs {
  unsigned char* ws;            // the absorbed-mode workspace
  AbsorbLayout lay;
  const void* Wk; const void* Wv; const void* bv;     // predictors of the layer ([D - m][D + m]), V bias or null
  // rotated keys (a.rope set), where the K side is explicit: the K predictor and bias the tensor-core kernel reads
  // -- where m splits a head, extended by the rows that pass the split head's stored dims through (kernels.h,
  // ReconArgs::m_heads) -- and the flat dims of the whole retained heads (-1: m)
  const void* Wk_x = nullptr; const void* bk_x = nullptr;
  int m_heads = -1;
  const void* bk = nullptr;     // K bias or null; read only when the keys are rotated (a.rope set): it cancels otherwise
  const void* bk_shift = nullptr;   // K bias or null: un-rotated keys with sink / window tokens, against whose true keys
                                    // the predicted tokens' scores are shifted by q . b_k
  int D, m;
  int capacity_tokens;
  bool save_k = false;          // the layer keeps its keys whole (k_local: pool of width D): no K predictor, every head's
                                // scores come from its stored keys; only the V side is predicted
  int n_sink = 0, n_window = 0; // sink / recent-window tokens kept at full precision (0, 0 = none) ...
  void* k_side = nullptr; void* v_side = nullptr;            // ... their dropped dims (side buffers of the layer)
  const void* k_local = nullptr; const void* v_local = nullptr;   // ... and the layer's pools (retained dims); also
                                                                 // read when the keys are rotated
  // rotated keys: the layer's K pool as the stored-head kernels see it (tensor maps in boxes of a page and of 64 rows)
  const CUtensorMap* k_stored = nullptr; const CUtensorMap* k_stored_run = nullptr;
  double* kernel_ms;            // unused
};

// One compressed layer, all query heads: out[B][H_q][d].  With a.rope set (keys cached before the rotary embedding) a
// rotation that depends on the token sits between Eq. 3 and q . k, so W_k cannot be folded into the queries: the K
// side is then explicit (predicted keys on the tensor cores, rotated, scored; stored heads scored from the pool)
// and only the V side uses the absorbed form.
cudaError_t launch_absorbed(const AttnArgs& a, const AbsorbArgs& r, const AbsorbMaps& maps, const TcLayerMaps& anchor,
                            const TcLayerMaps& layer, float* out, int sm_count, cudaStream_t stream,
                            cudaEvent_t* timing_events /* 4 events or null: around the K pass and the V pass */);

}  // namespace echokv
