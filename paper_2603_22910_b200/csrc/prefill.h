// Prefill-shaped attention (many queries per sequence): host interface of the row gather and the attention kernels.
#pragma once

#include "kernels.h"

namespace echokv {

// Stored dims 0 .. copy_width-1 (whole heads of 128, bf16) of every cached token, from a paged pool whose rows hold
// `width` dims into contiguous rows out[b][token][out_width]; keys are rotated to their positions if `rotate` and
// a.rope is set.  zero_tail > 0 also writes zeros over the whole rows len .. (next multiple of zero_tail) - 1
// (launched even when copy_width is 0).
cudaError_t launch_gather_rows(const AttnArgs& a, const void* pool, int width, int copy_width, __nv_bfloat16* out,
                               int out_tokens, int out_width, bool rotate, int zero_tail, cudaStream_t stream);

// Eq. 7 for n_q queries per sequence (a.q: [B][n_q][H_q][128] bf16), query i at position len - n_q + i attending the
// keys up to its own, over k_rows / v_rows [B][kv_tokens][kv_width] bf16.  out: fp32 [B][n_q][H_q][128].
// A sequence with fewer than n_q cached tokens gets zeros and the device status EBADLENGTH.
// path: 0 = mma.sync kernel, 1 = tcgen05 kernel (one thread group does every step in turn), 2 = warp-specialised
// tcgen05 kernel (needs v_rows zeroed from each sequence's length to the next multiple of 128 rows).
cudaError_t launch_prefill_attn(const AttnArgs& a, const __nv_bfloat16* k_rows, const __nv_bfloat16* v_rows,
                                int kv_tokens, int kv_width, int n_q, float* out, cudaStream_t stream, int path);

}  // namespace echokv
