// Tensor-core (tcgen05 / TMEM / TMA) reconstruct-then-attend path: host interface.
#pragma once

#include <cuda.h>

#include "kernels.h"

namespace echokv {

// TMA descriptors of one layer: its K and V pools (boxes of one page x 64 features) and, for a
// compressed layer, its two predictors (boxes of 256 rows x 64 input features).
struct TcLayerMaps {
  CUtensorMap k_pool, v_pool, wk, wv;
  CUtensorMap k_pool_run, v_pool_run;   // the pools again, in boxes of 64 token rows (runs of consecutive pages)
  // CTA-pair kernel: three-dimensional views [64-column chunk][row][64] whose boxes hold two chunks of
  // 128 rows each: of the pools (128 consecutive token rows) and of the predictors (one head)
  CUtensorMap k_pool_run128, v_pool_run128;
  CUtensorMap wk_half, wv_half;
  CUtensorMap wk_head, wv_head;         // the predictors in boxes of one head (128 rows) x 64 input features
  // CTA-pair kernel: the pools seen as [8-row group][64-column chunk][row of the group][64], so that ONE box holds
  // two 64-feature chunks of a page (or of a run of 64 / 128 consecutive token rows) and lands in shared memory as
  // 8-row swizzle atoms in the order (group, chunk): the groups of one chunk are then a uniform 2 KiB apart, which a
  // tensor-core operand descriptor can walk.  Boxes of one page, of 64 rows and of 128 rows
  CUtensorMap k_grp_page, k_grp_64, k_grp_128;
  CUtensorMap v_grp_page, v_grp_64, v_grp_128;
  CUtensorMap v_pool_tok64x4;           // [chunk][row][64] view of the V pool, boxes of 4 chunks x 64 rows
  bool pools_ready = false;
  bool weights_ready = false;
};

// TMA descriptor of a bf16 pool [rows][width]: boxes of box_rows token rows x 64 features, 128-byte swizzle.
cudaError_t encode_pool_box_map(CUtensorMap* map, const void* pool, int width, uint64_t rows, int box_rows);

// A bf16 pool [rows][width] seen as [rows / 8][width / 64][8][64] (8-row groups outermost): a box of box_rows rows x
// two 64-column chunks lands in shared memory as 1 KiB swizzle atoms (8 rows x 64 columns) in the order (group,
// chunk) -- one copy per page for both chunks of a head or of a stage.  A chunk past the last column reads as zeros.
cudaError_t encode_pool_group_map(CUtensorMap* map, const void* pool, int width, uint64_t rows, int box_rows);

// The matrix [rows][cols] seen as [cols / 64][rows][64]: boxes of box_chunks x box_rows x 64 land in shared
// memory as box_chunks consecutive swizzled sub-tiles of box_rows rows.
cudaError_t encode_chunked_3d_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, int box_rows,
                                  int box_chunks);

// General form: a bf16 tensor of `rank` dims (2..5, innermost first; strides in bytes for dims 1 .. rank-1), boxes in
// the 128-byte swizzle (innermost box extent 64 elements); elements outside the tensor read as zero.
cudaError_t encode_tiled_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                              const uint64_t* strides, const uint32_t* box);

bool tc_shape_supported(int dtype, int head_dim, int page_tokens, int D, int m);

// One small block that waits, with the kernels' own bounded-wait routine and a limit of limit_cycles, on a barrier
// nothing arrives on: raises ECHOKV_ETIMEOUT in *status and returns.  left_by[2] (device): how its two waiting warps
// left (1 = gave up / was released by the abort flag).
cudaError_t launch_bounded_wait_probe(int32_t* status, long long limit_cycles, int* left_by, cudaStream_t stream);

// k_width / v_width: row widths of the two pools (they differ where a layer keeps its keys whole); 0 = no pool
cudaError_t tc_encode_pool_maps(TcLayerMaps* maps, const void* k_pool, int k_width, const void* v_pool, int v_width,
                                uint64_t rows, int page_tokens);

cudaError_t tc_encode_weight_maps(TcLayerMaps* maps, const void* Wk, const void* Wv, int d_drop,
                                  int d_in);

// Dropped heads of one compressed layer: Eq. 3 on the tensor cores, Eq. 7 on the accumulators.
cudaError_t launch_recon_tc(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                            const TcLayerMaps& layer, int sm_count, cudaStream_t stream);

// The same on pairs of CTAs (cta_group::2, M = 256): one split-K partial per kPairPartTokens tokens.
cudaError_t launch_recon_pair(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                              const TcLayerMaps& layer, int sm_count, cudaStream_t stream);

// The same with four dropped heads per work item (a token tile is staged once per four heads; all of tensor memory
// belongs to the running phase): for long contractions with one or two query heads per KV head.
bool recon_quad_supported(int group);
cudaError_t launch_recon_quad(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                              const TcLayerMaps& layer, int sm_count, cudaStream_t stream);

// The K half of the same kernel for rotated keys (a.rope must be set): Eq. 3 for the dropped heads' keys, the
// rotation, q . k -- and the scores go to scores[b][query head][l_cap] (base-2 units; token slots that hold no
// predicted token get -inf, whole 256-token tiles are written) instead of into a softmax.  The V side is then
// evaluated with absorbed predictors.
cudaError_t launch_recon_pair_key_scores(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                                         const TcLayerMaps& layer, float* scores, int l_cap, int sm_count,
                                         cudaStream_t stream);

// Eq. 3 alone: the predicted dims of every cached token written out as 16-bit rows, out[b][token][out_width] at flat
// dims m .. D-1 (keys: bf16, + bias r.bk, rotated to the token's position if a.rope is set; values: fp16, the V
// predictor over the V pools; r.bk is then the V bias or null).  For uses with many queries per sequence, where rebuilding the
// cache once and attending it with a standard kernel is cheaper than rebuilding it per query.
cudaError_t launch_recon_pair_store(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                                    const TcLayerMaps& layer, bool values, __nv_bfloat16* out, int out_tokens,
                                    int out_width, int sm_count, cudaStream_t stream);

constexpr int kPairPartTokens = 128;

}  // namespace echokv
