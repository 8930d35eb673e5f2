// Prefill-shaped attention (many queries per sequence): host interface of the row gather and the attention kernels.
#pragma once

#include "kernels.h"

namespace echokv {

// Stored dims 0 .. copy_width-1 (whole heads of 128, bf16) of every cached token, from a paged pool whose rows hold
// `width` dims into contiguous rows out[b][token][out_width]; keys are rotated to their positions if `rotate` and
// a.rope is set.  zero_tail > 0 also writes zeros over the whole rows len .. (next multiple of zero_tail) - 1
// (launched even when copy_width is 0).
// to_half: the rows are written as fp16 instead (the value rows of the attention kernel below).
cudaError_t launch_gather_rows(const AttnArgs& a, const void* pool, int width, int copy_width, __nv_bfloat16* out,
                               int out_tokens, int out_width, bool rotate, int zero_tail, cudaStream_t stream,
                               bool to_half = false);

// Eq. 7 for n_q queries per sequence (a.q: [B][n_q][H_q][128] bf16), query i at position len - n_q + i attending the
// keys n_skip .. its own position - shift (plain causal attention: shift = n_skip = 0), over k_rows (bf16) and v_rows
// (fp16), [B][kv_tokens][kv_width] each (v_rows zeroed from each sequence's length to the next multiple of 128 rows).
// out: fp32 [B][n_q][H_q][128]; lse_out (may be null): fp32 [B][n_q][H_q], log2 of every row's softmax denominator in
// base-2 score units, -inf for a row that attends nothing (its output is zero).
// A sequence with fewer than n_q cached tokens gets zeros and the device status EBADLENGTH.
cudaError_t launch_prefill_attn(const AttnArgs& a, const __nv_bfloat16* k_rows, const __nv_bfloat16* v_rows,
                                int kv_tokens, int kv_width, int n_q, float* out, cudaStream_t stream, int shift = 0,
                                int n_skip = 0, float* lse_out = nullptr);

// The sink and recent-window tokens of every query at full precision (Section 4.1), added to what launch_prefill_attn
// (shift = n_window, n_skip = n_sink) left in out / lse: query i at position p reads the sink tokens t < min(n_sink,
// p + 1) from the layer's pools (dims below mk / m) and side buffers (the rest), and the window tokens
// max(n_sink, p - n_window + 1) .. p from k_recent / v_recent: [B][n_q + n_window - 1][D] bf16, whole K / V rows of
// the positions len - n_q - n_window + 1 .. len - 1 (rows of negative positions are never read).
struct PrefillBand {
  const void* k_recent; const void* v_recent;
  const void* k_pool; const void* v_pool;    // the layer's pools, row widths mk and m (null when 0)
  const void* k_side; const void* v_side;    // [max_batch][n_sink + n_window][D - m]; k_side null when mk == D
  int D, mk, m, d_drop, n_sink, n_window;
};
cudaError_t launch_prefill_band(const AttnArgs& a, const PrefillBand& band, int n_q, float* out, const float* lse,
                                cudaStream_t stream);

}  // namespace echokv
