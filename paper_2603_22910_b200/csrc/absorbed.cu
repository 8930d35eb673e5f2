// Absorbed-predictor decode of a compressed layer (bf16, head_dim 128).
//
// Eq. 3 is linear, so Eq. 7 over predicted heads needs neither K_hat nor V_hat:
//     q . (W_k x_t)           = (W_k^T q) . x_t            "absorbed query"  q~ = W_k^T q
//     sum_t p_t (W_v x_t)     = W_v (sum_t p_t x_t)         project after the weighted sum
// with x_t = [anchor dims ; retained dims] of token t (D_in values).  A retained head fits the
// same form with a q~ that selects its own dims, so all H_q query heads attend over the same
// per-token vectors and the layer becomes two streams over the cache plus small projections:
//
//   1. absorb_query_kernel   q~[b][h][:] for every head, scaled, split into two bf16 halves
//   2. absorb_scores_kernel  S[b][h][t] = q~ . x^K_t        tcgen05: M = 128 tokens, N = 2 H_q, K = D_in
//   3. absorb_softmax_kernel (max, sum) per head and token range; p = 2^(S - max of the range) as two bf16 halves
//   4. absorb_pv_kernel      y[b][h][:] = sum_t p_t x^V_t   tcgen05: M = 128 features (the V tile
//                            is the M-major A operand), N = 2 H_q, K = tokens; split over token
//                            ranges and 256-feature slices
//   5. absorb_ysum_kernel    y of the ranges merged by log-sum-exp and divided by the softmax sum;
//      absorb_out_kernel     out = W_v y (+ b_v) for predicted heads, y's own dims for retained heads
//
// The same result as the explicit path (Eq. 3, 6, 7) up to rounding, at 4 D_in bytes and
// 8 H_q D_in FLOP per token instead of 4 D_in D_drop FLOP: the two tcgen05 kernels are HBM-bound.
// Every wait is bounded.
#include "absorbed.h"

#include "stored_mma.h"

#include <cudaTypedefs.h>

#include "ptx_sm100.cuh"

namespace echokv {

namespace {

constexpr int kChunk = 64;
constexpr int kRowBytes = 128;
constexpr int kMaxStages = 6;
constexpr int kThreads = 256;            // warp 0 TMA, 1 MMA, 2 helper, 3 second TMA warp (V pass), 4..7 epilogue
constexpr int kMaxBatchPerLaunch = 256;
constexpr int kRunTokens = 64;
constexpr int kSmemBudget = 200 * 1024;

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ bool epi_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(ok ? 1u : 0u)
      : "memory");
  return r != 0;
}

// K-major bf16 operand: 128-byte rows in the 128-byte swizzle, 8-row groups group_bytes apart
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t smem_addr, uint32_t group_bytes = 1024) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(group_bytes >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// M-major bf16 operand made of [K rows][64 M-elements] tiles in the 128-byte swizzle (what a TMA box
// of token rows x 64 features is when tokens are the contraction index): 8-row groups along K are
// group_bytes apart, successive 64-element blocks along M are `block_bytes` apart
__device__ __forceinline__ uint64_t desc_mmajor(uint32_t smem_addr, uint32_t block_bytes, uint32_t group_bytes = 1024) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);
  d |= static_cast<uint64_t>(block_bytes >> 4) << 16;
  d |= static_cast<uint64_t>(group_bytes >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// kind::f16, bf16 x bf16 -> fp32, M = 128; a_mmajor: the A operand is M-major (B always K-major)
inline uint32_t make_idesc(int n, bool a_mmajor) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (a_mmajor ? (1u << 15) : 0u) | ((uint32_t)(n >> 3) << 17) |
         ((128u >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------
// 1. absorbed queries
// ---------------------------------------------------------------------------------------------
constexpr int kQGroup = 8;   // (sequence, query head of the group) pairs per block
constexpr int kQCols = 256;  // input features per block: eight adjacent ones per lane
constexpr size_t kQuerySmemBytes = (size_t)(kQGroup * 128 + 8 * kQGroup * kQCols) * sizeof(float);

// Block = (256 input features, KV head, 8 (sequence, query head) pairs).  The head's predictor rows are dealt
// round-robin to the 8 warps, each lane reading 16 bytes (8 features) of a row, so a thread has all its
// loads in flight at once; the warps' partial sums meet in shared memory.
__global__ void __launch_bounds__(256)
absorb_query_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ Wk,
                    __nv_bfloat16* __restrict__ q2, int B, int n_q_heads, int g, int m, int D, int d_in,
                    float scale_log2e) {
  extern __shared__ __align__(16) float query_smem[];
  float (*qs)[128] = reinterpret_cast<float (*)[128]>(query_smem);          // [kQGroup][128]
  float* red = query_smem + kQGroup * 128;                                  // [8 warps][kQGroup][kQCols]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col0 = blockIdx.x * kQCols;
  const int kv = blockIdx.y;
  const int first = blockIdx.z * kQGroup;
  const int n_pairs = B * g;
  for (int idx = tid; idx < kQGroup * 128; idx += 256) {
    const int k = idx >> 7, j = idx & 127;
    const int pr = first + k;
    float v = 0.f;
    if (pr < n_pairs) {
      const int b = pr / g, gi = pr - b * g;
      v = __bfloat162float(q[((size_t)b * n_q_heads + kv * g + gi) * 128 + j]) * scale_log2e;
    }
    qs[k][j] = v;
  }
  __syncthreads();
  // dims kv * 128 + j of this head with flat index < m are stored (the head reads them as they are: q~ is q
  // placed at those local dims); the others are predicted by row (flat index - m) of W_k
  const int n_stored = max(0, min(128, m - kv * 128));
  float acc[kQGroup][8];
#pragma unroll
  for (int k = 0; k < kQGroup; ++k)
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[k][c] = 0.f;
  const int i8 = col0 + lane * 8;                    // this lane's eight input features (d_in is a multiple of 8)
  if (i8 < d_in && n_stored < 128) {
    const __nv_bfloat16* w = Wk + (size_t)(kv * 128 + n_stored + warp - m) * d_in + i8;
#pragma unroll 8
    for (int j = n_stored + warp; j < 128; j += 8, w += (size_t)8 * d_in) {
      const uint4 raw = *reinterpret_cast<const uint4*>(w);
      const uint32_t r4[4] = {raw.x, raw.y, raw.z, raw.w};
      float wv[8];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        wv[2 * c] = __uint_as_float(r4[c] << 16);
        wv[2 * c + 1] = __uint_as_float(r4[c] & 0xffff0000u);
      }
#pragma unroll
      for (int k = 0; k < kQGroup; ++k) {
        const float qv = qs[k][j];
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[k][c] = fmaf(wv[c], qv, acc[k][c]);
      }
    }
  }
#pragma unroll
  for (int k = 0; k < kQGroup; ++k) {
    float4* dst = reinterpret_cast<float4*>(red + (size_t)(warp * kQGroup + k) * kQCols + lane * 8);
    dst[0] = make_float4(acc[k][0], acc[k][1], acc[k][2], acc[k][3]);
    dst[1] = make_float4(acc[k][4], acc[k][5], acc[k][6], acc[k][7]);
  }
  __syncthreads();
  const int i = col0 + tid;                          // one input feature per thread from here on
  if (i >= d_in) return;
  const int j_stored = i - (D + kv * 128);
  const int nh2 = 2 * n_q_heads;
#pragma unroll
  for (int k = 0; k < kQGroup; ++k) {
    const int pr = first + k;
    if (pr >= n_pairs) break;
    float v = (j_stored >= 0 && j_stored < n_stored) ? qs[k][j_stored] : 0.f;
#pragma unroll
    for (int w8 = 0; w8 < 8; ++w8) v += red[(size_t)(w8 * kQGroup + k) * kQCols + tid];
    const int b = pr / g, gi = pr - b * g;
    const int h = kv * g + gi;
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    q2[((size_t)b * nh2 + h) * d_in + i] = hi;
    q2[((size_t)b * nh2 + n_q_heads + h) * d_in + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
  }
}

// ---------------------------------------------------------------------------------------------
// shared pieces of the two tcgen05 kernels
// ---------------------------------------------------------------------------------------------
struct StreamParams {
  const int32_t* slots;
  const int32_t* lens;
  const int32_t* table;
  int max_batch, max_pages_per_seq, page_tokens;
  long long n_pages;
  int32_t* status;
  int b0, nb;
  int n_q_heads, nh2;
  int kc_anchor, kc_total;      // 64-feature chunks: from the anchor pool, in all
  int run_pages;                // pages per 64-row run box, 1 = none
  int l_cap;
  int n_stages;
  uint32_t stage_bytes;
  uint32_t idesc;
  float* s_out;                 // scores kernel: S
  float* y_out;                 // pv kernel: partial y
  int d_in;
  int range_tokens;             // pv kernel: tokens per range
  int n_slices;                 // pv kernel: 256-feature slices
  int n_sink, n_window;         // scores kernel: sink / recent-window tokens are left to the side kernel
};

struct StreamSmemTail {
  int cum[kMaxBatchPerLaunch + 1];
  unsigned long long full_bar[kMaxStages];
  unsigned long long empty_bar[kMaxStages];
  unsigned long long clean_bar[kMaxStages];
  unsigned long long acc_full_bar[2];
  unsigned long long acc_empty_bar[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ int find_seq(const StreamSmemTail& t, int unit, int nb) {
  int lo = 0, hi = nb;   // largest b with cum[b] <= unit
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (t.cum[mid] <= unit) lo = mid; else hi = mid;
  }
  return lo;
}

// Per-sequence unit counts -> exclusive prefix sums in t.cum; barriers; tensor memory.
template <typename CountFn>
__device__ __forceinline__ void stream_setup(StreamSmemTail& t, const StreamParams& p, uint32_t tmem_cols,
                                             CountFn count) {
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int i = tid; i < p.nb; i += kThreads) {
    const int b = p.b0 + i;
    const int slot = p.slots ? p.slots[b] : b;
    const int len = p.lens[b];
    int n = 0;
    if (slot < 0 || slot >= p.max_batch) {
      if (blockIdx.x == 0) report(p.status, ECHOKV_EBADPAGE);
    } else if (len < 1 || len > p.max_pages_per_seq * p.page_tokens) {
      if (blockIdx.x == 0) report(p.status, ECHOKV_EBADLENGTH);
    } else {
      n = count(len);
    }
    t.cum[i + 1] = n;
  }
  if (tid == 0) {
    t.cum[0] = 0;
    t.abort_flag = 0;
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(smem_u32(&t.full_bar[s]), 1);
      mbar_init(smem_u32(&t.empty_bar[s]), 1);
      mbar_init(smem_u32(&t.clean_bar[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&t.acc_full_bar[i]), 1);
      mbar_init(smem_u32(&t.acc_empty_bar[i]), 1);
    }
    mbar_fence_init();
  }
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int i = 0; i < p.nb; ++i) {
      acc += t.cum[i + 1];
      t.cum[i + 1] = acc;
    }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&t.tmem_base), tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
}

// The `n_boxes` boxes of `box_tokens` token rows (a page, or part of a page when pages are taller than the
// span wanted) that start at token t0 of the sequence in block-table row `slot`: lane i holds the pool row
// where box i starts (-1 = no cached token there or a bad page id); whether the boxes form one
// consecutive run in the pool; and for 64-row sub-runs which lane leads / follows.
struct PageSet {
  int row;
  bool all_run;        // every box valid and consecutive in the pool
  bool run_lead, run_member;
  uint32_t n_valid;
};
// Block-table entry of box `lane` (only the load: callers may issue it a stage ahead of its use)
__device__ __forceinline__ int load_page(const StreamParams& p, int slot, int len, int t0, int n_boxes,
                                         int box_tokens, int lane) {
  const int tb = t0 + lane * box_tokens;
  if (lane < n_boxes && tb < len) return p.table[(size_t)slot * p.max_pages_per_seq + tb / p.page_tokens];
  return -1;
}
__device__ __forceinline__ PageSet make_page_set(const StreamParams& p, int raw_page, int len, int t0, int n_boxes,
                                                 int box_tokens, int lane) {
  PageSet r;
  r.row = -1;
  const int tb = t0 + lane * box_tokens;
  if (lane < n_boxes && tb < len) {
    if (raw_page < 0 || raw_page >= p.n_pages) report(p.status, ECHOKV_EBADPAGE);
    else r.row = raw_page * p.page_tokens + tb % p.page_tokens;
  }
  r.n_valid = __popc(__ballot_sync(0xffffffffu, r.row >= 0));
  const int row0 = __shfl_sync(0xffffffffu, r.row, 0);
  r.all_run = __all_sync(0xffffffffu, lane >= n_boxes || (r.row >= 0 && r.row == row0 + lane * box_tokens));
  r.run_lead = r.run_member = false;
  if (p.run_pages > 1) {
    bool consecutive = r.row >= 0;
    for (int k = 1; k < p.run_pages; ++k) {
      const int rk = __shfl_down_sync(0xffffffffu, r.row, k);
      consecutive = consecutive && rk == r.row + k * box_tokens;
    }
    const int lead = lane - lane % p.run_pages;
    const bool group_run = __shfl_sync(0xffffffffu, consecutive ? 1 : 0, lead) != 0;
    r.run_lead = group_run && lane == lead && lane < n_boxes;
    r.run_member = group_run && lane != lead && lane < n_boxes;
  }
  return r;
}
__device__ __forceinline__ PageSet lookup_pages(const StreamParams& p, int slot, int len, int t0, int n_boxes,
                                                int box_tokens, int lane) {
  return make_page_set(p, load_page(p, slot, len, t0, n_boxes, box_tokens, lane), len, t0, n_boxes, box_tokens, lane);
}

// ---------------------------------------------------------------------------------------------
// 2. scores: S[b][h][t] = q~[b][h] . x^K_t
// ---------------------------------------------------------------------------------------------
constexpr int kScoreTokens = 128;                    // tokens per work item
constexpr int kScoreXBytes = kScoreTokens * kRowBytes;   // one chunk of the token rows

__global__ void __launch_bounds__(kThreads, 1)
absorb_scores_kernel(const __grid_constant__ CUtensorMap tm_anchor, const __grid_constant__ CUtensorMap tm_local,
                     const __grid_constant__ CUtensorMap tm_anchor_run, const __grid_constant__ CUtensorMap tm_local_run,
                     const __grid_constant__ CUtensorMap tm_anchor_128, const __grid_constant__ CUtensorMap tm_local_128,
                     const __grid_constant__ CUtensorMap tm_q2, const StreamParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  StreamSmemTail& t = *reinterpret_cast<StreamSmemTail*>(smem + (size_t)p.n_stages * p.stage_bytes);
  const uint32_t stage_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &t.abort_flag;
  stream_setup(t, p, 256u, [](int len) { return (len + kScoreTokens - 1) / kScoreTokens; });
  const uint32_t tmem = t.tmem_base;
  const int n_items = t.cum[p.nb];
  const int n_steps = (p.kc_total + 1) / 2;               // stages per item: two chunks each (the last maybe one)
  const int box_tokens = min(p.page_tokens, kScoreTokens);
  const int boxes = kScoreTokens / box_tokens;
  const uint32_t page_bytes = box_tokens * kRowBytes;
  const uint32_t q_chunk_bytes = (uint32_t)p.nh2 * kRowBytes;

  if (warp == 0 || warp == 3) {
    // =============================== TMA producers (alternate stages) ===========================
    const uint32_t mine = warp == 0 ? 0u : 1u;
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const int bi = find_seq(t, item, p.nb);
      const int b = p.b0 + bi;
      const int tile = item - t.cum[bi];
      const int slot = p.slots ? p.slots[b] : b;
      const int len = p.lens[b];
      const PageSet ps = lookup_pages(p, slot, len, tile * kScoreTokens, boxes, box_tokens, lane);
      for (int step = 0; step < n_steps; ++step, ++it) {
        if ((it & 1u) != mine) continue;
        const uint32_t s = it % p.n_stages;
        const uint32_t ph = (it / p.n_stages) & 1u;
        const uint32_t full = smem_u32(&t.full_bar[s]);
        bool ok = true;
        if (lane == 0) ok = mbar_wait(smem_u32(&t.empty_bar[s]), ph ^ 1u, abort_flag, p.status);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) { alive = false; break; }
        const int kc0 = step * 2;                           // both chunks come from the same pool
        const int n_chunks = min(2, p.kc_total - kc0);
        const bool from_anchor = kc0 < p.kc_anchor;
        const int kx0 = from_anchor ? kc0 : kc0 - p.kc_anchor;
        // (every box brings two chunks -- of the token rows as (8-row group, chunk) swizzle atoms, one copy per page
        // for both -- and so does the absorbed-query box: past the last chunk they are filled with zeros)
        if (lane == 0) mbar_arrive_expect_tx(full, 2u * ps.n_valid * page_bytes + 2u * q_chunk_bytes);
        __syncwarp();
        const uint32_t x_dst = stage_base + s * p.stage_bytes;
        if (ps.all_run) {
          if (lane == 0)
            tma_load_4d(x_dst, from_anchor ? &tm_anchor_128 : &tm_local_128, 0, 0, kx0, ps.row >> 3, full);
        } else if (ps.row >= 0 && !ps.run_member) {
          const CUtensorMap* m = ps.run_lead ? (from_anchor ? &tm_anchor_run : &tm_local_run)
                                             : (from_anchor ? &tm_anchor : &tm_local);
          tma_load_4d(x_dst + lane * 2 * page_bytes, m, 0, 0, kx0, ps.row >> 3, full);
        }
        if (lane == 16) tma_load_3d(x_dst + 2 * kScoreXBytes, &tm_q2, 0, b * p.nh2, kc0, full);
      }
    }
  } else if (warp == 1) {
    // =============================== MMA issuer ================================================
    if (lane == 0) {
      uint32_t it = 0, n = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x, ++n) {
        const uint32_t buf = n & 1u;
        if (!mbar_wait(smem_u32(&t.acc_empty_bar[buf]), ((n >> 1) & 1u) ^ 1u, abort_flag, p.status)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem + buf * 128u;
        for (int step = 0; step < n_steps; ++step, ++it) {
          const uint32_t s = it % p.n_stages;
          const uint32_t ph = (it / p.n_stages) & 1u;
          if (!mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status)) { alive = false; break; }
          tc_fence_after();
          const uint32_t x_addr = stage_base + s * p.stage_bytes;
          const int n_chunks = min(2, p.kc_total - step * 2);
          for (int j = 0; j < n_chunks; ++j) {
            const uint64_t a_desc = desc_kmajor(x_addr + j * 1024, 2048);     // groups of one chunk: 2 KiB apart
            const uint64_t b_desc = desc_kmajor(x_addr + 2 * kScoreXBytes + j * q_chunk_bytes);
#pragma unroll
            for (int k16 = 0; k16 < 4; ++k16)
              tc_mma_bf16(d_tmem, a_desc + 2 * k16, b_desc + 2 * k16, p.idesc, (step > 0 || j > 0 || k16 > 0) ? 1u : 0u);
          }
          tc_commit(smem_u32(&t.empty_bar[s]));
        }
        if (alive) tc_commit(smem_u32(&t.acc_full_bar[buf]));
      }
    }
    __syncwarp();
  } else if (warp >= 4) {
    // =============================== epilogue (4 warps) ========================================
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;                 // TMEM lane = token of the tile
    uint32_t n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const int bi = find_seq(t, item, p.nb);
      const int b = p.b0 + bi;
      const int tile = item - t.cum[bi];
      const int len = p.lens[b];
      const uint32_t buf = n & 1u;
      if (!epi_all(mbar_wait(smem_u32(&t.acc_full_bar[buf]), (n >> 1) & 1u, abort_flag, p.status))) break;
      tc_fence_after();
      const int token = tile * kScoreTokens + row;
      const bool valid = token >= predicted_lo(len, p.n_sink) && token < predicted_hi(len, p.n_sink, p.n_window);
      const uint32_t addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 128u;
      float* dst = p.s_out + (size_t)b * p.n_q_heads * p.l_cap + token;
      for (int hb = 0; hb < p.n_q_heads; hb += 16) {
        float hi[16], lo[16];
        tmem_ld16(addr + hb, hi);
        tmem_ld16(addr + p.n_q_heads + hb, lo);
#pragma unroll
        for (int k = 0; k < 16; ++k)
          dst[(size_t)(hb + k) * p.l_cap] = valid ? hi[k] + lo[k] : -INFINITY;
      }
      tc_fence_before();
      epi_sync();
      if (tid == 128) mbar_arrive(smem_u32(&t.acc_empty_bar[buf]));
    }
  }

  if (t.abort_flag) {     // a wait ran out: give copies and MMAs already started ample time to land
    const long long start = clock64();
    while (clock64() - start < 4000000ll) {
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 256u);
  }
}

// ---------------------------------------------------------------------------------------------
// 3. softmax statistics and probabilities
// ---------------------------------------------------------------------------------------------
// One block per (query head, sequence, token range of the V pass): the range's own maximum and sum, and its
// probabilities relative to that maximum; the ranges are merged by log-sum-exp in absorb_ysum_kernel.
__global__ void __launch_bounds__(256)
absorb_softmax_kernel(const float* __restrict__ S, __nv_bfloat16* __restrict__ p2, float2* __restrict__ ml_range,
                      const int32_t* __restrict__ slots, const int32_t* __restrict__ lens, int max_batch,
                      int capacity, int n_q_heads, int l_cap, int range_tokens) {
  const int h = blockIdx.x, b = blockIdx.y, range = blockIdx.z, tid = threadIdx.x;
  const int slot = slots ? slots[b] : b;
  const int len = lens[b];
  if (slot < 0 || slot >= max_batch || len < 1 || len > capacity) return;   // (absorb_ysum_kernel writes zeros)
  const int t_begin = range * range_tokens;
  if (t_begin >= len) return;
  const int t_end = min(len, t_begin + range_tokens);
  __shared__ float red[8];
  const float* s = S + ((size_t)b * n_q_heads + h) * l_cap + t_begin;
  const int n4 = (t_end - t_begin + 3) / 4;      // (entries past len hold -inf up to the next 128)
  float m = -INFINITY;
  for (int i = tid; i < n4; i += 256) {
    const float4 v = reinterpret_cast<const float4*>(s)[i];
    m = fmaxf(fmaxf(m, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
  }
  m = warp_max(m);
  if ((tid & 31) == 0) red[tid >> 5] = m;
  __syncthreads();
  float M = red[0];
#pragma unroll
  for (int w = 1; w < 8; ++w) M = fmaxf(M, red[w]);
  __syncthreads();
  const float M_out = M;
  if (M == -INFINITY) M = 0.f;     // every token of the range is a sink / window token: all probabilities are 0
  const int nh2 = 2 * n_q_heads;
  __nv_bfloat16* hi = p2 + ((size_t)b * nh2 + h) * l_cap + t_begin;
  __nv_bfloat16* lo = p2 + ((size_t)b * nh2 + n_q_heads + h) * l_cap + t_begin;
  const int n4_pad = ((t_end - t_begin + 63) / 64) * 16;     // the V pass reads whole 64-token blocks
  float L = 0.f;
  for (int i = tid; i < n4_pad; i += 256) {
    const float4 v = reinterpret_cast<const float4*>(s)[i];
    const float pv[4] = {exp2f(v.x - M), exp2f(v.y - M), exp2f(v.z - M), exp2f(v.w - M)};   // 2^(-inf) = 0
    L += (pv[0] + pv[1]) + (pv[2] + pv[3]);
    const __nv_bfloat162 h01 = __floats2bfloat162_rn(pv[0], pv[1]);
    const __nv_bfloat162 h23 = __floats2bfloat162_rn(pv[2], pv[3]);
    const __nv_bfloat162 l01 = __floats2bfloat162_rn(pv[0] - __low2float(h01), pv[1] - __high2float(h01));
    const __nv_bfloat162 l23 = __floats2bfloat162_rn(pv[2] - __low2float(h23), pv[3] - __high2float(h23));
    uint2 uh, ul;
    uh.x = *reinterpret_cast<const uint32_t*>(&h01); uh.y = *reinterpret_cast<const uint32_t*>(&h23);
    ul.x = *reinterpret_cast<const uint32_t*>(&l01); ul.y = *reinterpret_cast<const uint32_t*>(&l23);
    reinterpret_cast<uint2*>(hi)[i] = uh;
    reinterpret_cast<uint2*>(lo)[i] = ul;
  }
  L = warp_sum(L);
  if ((tid & 31) == 0) red[tid >> 5] = L;
  __syncthreads();
  if (tid == 0) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) tot += red[w];
    ml_range[((size_t)b * n_q_heads + h) * kAbsorbMaxRanges + range] = make_float2(M_out, tot);
  }
}

// ---------------------------------------------------------------------------------------------
// 4. y[b][h][:] = sum_t p[b][h][t] x^V_t, per (sequence, token range, 256-feature slice)
// ---------------------------------------------------------------------------------------------
constexpr int kPvTokens = 64;                        // tokens per stage
constexpr int kPvTileBytes = kPvTokens * kRowBytes;  // 64 token rows x 64 features
constexpr int kPvVBytes = 4 * kPvTileBytes;          // four chunks

__global__ void __launch_bounds__(kThreads, 1)
absorb_pv_kernel(const __grid_constant__ CUtensorMap tm_anchor, const __grid_constant__ CUtensorMap tm_local,
                 const __grid_constant__ CUtensorMap tm_anchor_run, const __grid_constant__ CUtensorMap tm_local_run,
                 const __grid_constant__ CUtensorMap tm_p2, const StreamParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  StreamSmemTail& t = *reinterpret_cast<StreamSmemTail*>(smem + (size_t)p.n_stages * p.stage_bytes);
  const uint32_t stage_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &t.abort_flag;
  const int range_tokens = p.range_tokens, n_slices = p.n_slices;
  stream_setup(t, p, 512u, [range_tokens, n_slices](int len) {
    return ((len + range_tokens - 1) / range_tokens) * n_slices;
  });
  const uint32_t tmem = t.tmem_base;
  const int n_items = t.cum[p.nb];
  const int box_tokens = min(p.page_tokens, kPvTokens);     // (a taller page is read 64 rows at a time)
  const int boxes = kPvTokens / box_tokens;                 // boxes per chunk and stage
  const uint32_t page_bytes = box_tokens * kRowBytes;
  const uint32_t p_tile_bytes = (uint32_t)p.nh2 * kRowBytes;

  // item -> (sequence, range, slice); its token span and chunk span
  struct Work { int b, slot, len, range, slice, t_begin, n_steps, kc0, n_chunks; bool from_anchor; };
  auto decode = [&](int item) {
    Work w;
    const int bi = find_seq(t, item, p.nb);
    w.b = p.b0 + bi;
    const int local = item - t.cum[bi];
    w.range = local / n_slices;
    w.slice = local - w.range * n_slices;
    w.slot = p.slots ? p.slots[w.b] : w.b;
    w.len = p.lens[w.b];
    w.t_begin = w.range * range_tokens;
    const int t_end = min(w.len, w.t_begin + range_tokens);
    w.n_steps = (t_end - w.t_begin + kPvTokens - 1) / kPvTokens;
    w.kc0 = w.slice * 4;
    w.n_chunks = min(4, p.kc_total - w.kc0);
    w.from_anchor = w.kc0 < p.kc_anchor;   // (D / 64 is a multiple of 4 when the tiled maps are in use)
    return w;
  };

  if (warp == 0 || warp == 3) {
    // =============================== TMA producers ==============================================
    // Two warps take alternate stages: what one thread must do per stage (block-table entries, run
    // detection, two copies) is what limits a single producer here, not the memory system.
    const uint32_t mine = warp == 0 ? 0u : 1u;
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Work w = decode(item);
      // block-table entries are requested one own stage (two stages) ahead of their use
      const int first = ((it & 1u) == mine) ? 0 : 1;
      int raw_next = first < w.n_steps
                         ? load_page(p, w.slot, w.len, w.t_begin + first * kPvTokens, boxes, box_tokens, lane) : -1;
      for (int step = 0; step < w.n_steps; ++step, ++it) {
        if ((it & 1u) != mine) continue;
        const int raw = raw_next;
        if (step + 2 < w.n_steps)
          raw_next = load_page(p, w.slot, w.len, w.t_begin + (step + 2) * kPvTokens, boxes, box_tokens, lane);
        const uint32_t s = it % p.n_stages;
        const uint32_t ph = (it / p.n_stages) & 1u;
        const uint32_t full = smem_u32(&t.full_bar[s]);
        bool ok = true;
        if (lane == 0) ok = mbar_wait(smem_u32(&t.empty_bar[s]), ph ^ 1u, abort_flag, p.status);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) { alive = false; break; }
        const int t0 = w.t_begin + step * kPvTokens;
        const PageSet ps = make_page_set(p, raw, w.len, t0, boxes, box_tokens, lane);
        // The value rows of a stage are two 16 KiB halves (features 0-127 and 128-255 of the slice), each laid out
        // as (8-token group, chunk) swizzle atoms: one copy per page brings both chunks of a half (a chunk past the
        // end of the pool rows reads as zeros)
        const int n_mt = (w.n_chunks + 1) / 2;
        if (lane == 0) mbar_arrive_expect_tx(full, 2u * (uint32_t)n_mt * ps.n_valid * page_bytes + p_tile_bytes);
        __syncwarp();
        const uint32_t v_dst = stage_base + s * p.stage_bytes;
        for (int mt = 0; mt < n_mt; ++mt) {
          const int kc = w.kc0 + 2 * mt;                 // (a pair of chunks never straddles the two pools: D / 64 is even)
          const bool fa = kc < p.kc_anchor;
          const int kx = fa ? kc : kc - p.kc_anchor;
          if (ps.all_run) {
            if (lane == 0) tma_load_4d(v_dst + mt * 2 * kPvTileBytes, fa ? &tm_anchor_run : &tm_local_run, 0, 0, kx, ps.row >> 3, full);
          } else if (ps.row >= 0 && !ps.run_member) {
            // (pages of 64 tokens or more: the 64-row maps are the box of one stage)
            const bool tall = ps.run_lead || p.page_tokens >= kPvTokens;
            const CUtensorMap* m = tall ? (fa ? &tm_anchor_run : &tm_local_run) : (fa ? &tm_anchor : &tm_local);
            tma_load_4d(v_dst + mt * 2 * kPvTileBytes + lane * 2 * page_bytes, m, 0, 0, kx, ps.row >> 3, full);
          }
        }
        if (lane == 16) tma_load_2d(v_dst + kPvVBytes, &tm_p2, t0, w.b * p.nh2, full);
      }
    }
  } else if (warp == 1) {
    // =============================== MMA issuer ================================================
    if (lane == 0) {
      uint32_t it = 0, n = 0;
      uint32_t clean_uses[kMaxStages];
#pragma unroll
      for (int s = 0; s < kMaxStages; ++s) clean_uses[s] = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x, ++n) {
        const Work w = decode(item);
        const uint32_t buf = n & 1u;
        if (!mbar_wait(smem_u32(&t.acc_empty_bar[buf]), ((n >> 1) & 1u) ^ 1u, abort_flag, p.status)) break;
        tc_fence_after();
        const int n_mtiles = (w.n_chunks + 1) / 2;   // (a last tile may be half filled: its upper rows are unused)
        for (int step = 0; step < w.n_steps; ++step, ++it) {
          const uint32_t s = it % p.n_stages;
          const uint32_t ph = (it / p.n_stages) & 1u;
          if (!mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status)) { alive = false; break; }
          if (w.t_begin + (step + 1) * kPvTokens > w.len) {
            // a block with slots that hold no token: wait until the helper warp has zeroed them
            if (!mbar_wait(smem_u32(&t.clean_bar[s]), clean_uses[s] & 1u, abort_flag, p.status)) { alive = false; break; }
            ++clean_uses[s];
          }
          tc_fence_after();
          const uint32_t v_addr = stage_base + s * p.stage_bytes;
          const uint64_t b_desc = desc_kmajor(v_addr + kPvVBytes);
          for (int mt = 0; mt < n_mtiles; ++mt) {
            // A: 128 features (two 64-feature atoms, 1 KiB apart) x 16 tokens per MMA, M-major; 8-token groups 2 KiB apart
            const uint64_t a_desc = desc_mmajor(v_addr + mt * 2 * kPvTileBytes, 1024, 2048);
            const uint32_t d_tmem = tmem + buf * 256u + mt * (uint32_t)p.nh2;
#pragma unroll
            for (int k16 = 0; k16 < 4; ++k16)   // 16 tokens = two groups = 4096 bytes of A, 32 bytes along B's K
              tc_mma_bf16(d_tmem, a_desc + 256 * k16, b_desc + 2 * k16, p.idesc, (step > 0 || k16 > 0) ? 1u : 0u);
          }
          tc_commit(smem_u32(&t.empty_bar[s]));
        }
        if (alive) tc_commit(smem_u32(&t.acc_full_bar[buf]));
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ============ helper: zero V rows of slots that hold no token (never written, or a skipped page) ====
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Work w = decode(item);
      for (int step = 0; step < w.n_steps; ++step, ++it) {
        const uint32_t s = it % p.n_stages;
        const uint32_t ph = (it / p.n_stages) & 1u;
        const bool got = mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
        const int n_tok = w.len - (w.t_begin + step * kPvTokens);
        if (n_tok >= kPvTokens) continue;
        const uint32_t v_addr = stage_base + s * p.stage_bytes;
        const int n_rows = kPvTokens - n_tok;                 // rows n_tok .. 63 of every chunk tile
        for (int idx = lane; idx < w.n_chunks * n_rows * 8; idx += 32) {
          const int piece = idx & 7, rr = (idx >> 3) % n_rows, c = (idx >> 3) / n_rows;
          const int tr = n_tok + rr;            // (all eight pieces of the row are zeroed: the swizzle does not matter)
          const uint32_t a = v_addr + (c >> 1) * 2 * kPvTileBytes + (tr >> 3) * 2048 + (c & 1) * 1024 + (tr & 7) * kRowBytes +
                             piece * 16;
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0u) : "memory");
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&t.clean_bar[s]));
      }
    }
  } else if (warp >= 4) {
    // =============================== epilogue (4 warps) ========================================
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;                 // TMEM lane = feature of the 128-feature tile
    uint32_t n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const Work w = decode(item);
      const uint32_t buf = n & 1u;
      if (!epi_all(mbar_wait(smem_u32(&t.acc_full_bar[buf]), (n >> 1) & 1u, abort_flag, p.status))) break;
      tc_fence_after();
      const int n_mtiles = (w.n_chunks + 1) / 2;
      for (int mt = 0; mt < n_mtiles; ++mt) {
        const uint32_t addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 256u + mt * (uint32_t)p.nh2;
        const int feature = w.kc0 * kChunk + mt * 128 + row;
        if (feature >= p.d_in) continue;          // (rows of a half-filled tile that stand for no feature)
        float* dst = p.y_out + (((size_t)w.b * kAbsorbMaxRanges + w.range) * p.n_q_heads) * p.d_in + feature;
        for (int hb = 0; hb < p.n_q_heads; hb += 16) {
          float hi[16], lo[16];
          tmem_ld16(addr + hb, hi);
          tmem_ld16(addr + p.n_q_heads + hb, lo);
#pragma unroll
          for (int k = 0; k < 16; ++k) dst[(size_t)(hb + k) * p.d_in] = hi[k] + lo[k];
        }
      }
      tc_fence_before();
      epi_sync();
      if (tid == 128) mbar_arrive(smem_u32(&t.acc_empty_bar[buf]));
    }
  }

  if (t.abort_flag) {
    const long long start = clock64();
    while (clock64() - start < 4000000ll) {
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512u);
  }
}

// ---------------------------------------------------------------------------------------------
// 5. output: sum the ranges, normalise, project
// ---------------------------------------------------------------------------------------------
// ysum[b][h][i] = log-sum-exp merge over the sequence's ranges of y[b][range][h][i] (each relative to its
// range's maximum), divided by the merged softmax sum; ml[b][h] receives the merged (max, sum)
__global__ void __launch_bounds__(256)
absorb_ysum_kernel(const float* __restrict__ y, const float2* __restrict__ ml_range, float2* __restrict__ ml,
                   float* __restrict__ ysum, const int32_t* __restrict__ slots, const int32_t* __restrict__ lens,
                   int max_batch, int capacity, int n_q_heads, int d_in, int range_tokens) {
  const int h = blockIdx.y, b = blockIdx.z;
  const int i4 = blockIdx.x * 256 + threadIdx.x;        // float4 index inside the row
  const int slot = slots ? slots[b] : b;
  const int len = lens[b];
  const bool usable = slot >= 0 && slot < max_batch && len >= 1 && len <= capacity;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float M = -INFINITY, L = 0.f;
  if (usable) {
    const int n_ranges = (len + range_tokens - 1) / range_tokens;
    const float2* mr = ml_range + ((size_t)b * n_q_heads + h) * kAbsorbMaxRanges;
    for (int r = 0; r < n_ranges; ++r) M = fmaxf(M, mr[r].x);
    if (M > -INFINITY && i4 * 4 < d_in) {
      const float4* src = reinterpret_cast<const float4*>(y + (((size_t)b * kAbsorbMaxRanges) * n_q_heads + h) * d_in) + i4;
      const size_t range_stride4 = (size_t)n_q_heads * d_in / 4;
      for (int r = 0; r < n_ranges; ++r) {
        const float2 m = mr[r];
        const float w = exp2f(m.x - M);
        L = fmaf(w, m.y, L);
        const float4 v = src[r * range_stride4];
        acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
        acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
      }
      const float inv = L > 0.f ? 1.f / L : 0.f;
      acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    } else if (M > -INFINITY) {
      for (int r = 0; r < n_ranges; ++r) L = fmaf(exp2f(mr[r].x - M), mr[r].y, L);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) ml[(size_t)b * n_q_heads + h] = make_float2(M, L);
  if (i4 * 4 < d_in) reinterpret_cast<float4*>(ysum + ((size_t)b * n_q_heads + h) * d_in)[i4] = acc;
}

constexpr int kOutRows = 16;     // output features per block
constexpr int kOutPairs = 8;     // (sequence, query head of the group) pairs per block

// out[b][h][j] = W_v[row of (kv, j)] . ysum[b][h]  (+ b_v) for predicted heads; ysum's own dims for retained
// heads.  A block takes 16 output features x 8 (sequence, head) pairs; its 8 warps split the contraction,
// so every y value loaded is used for all 16 rows.
__global__ void __launch_bounds__(256)
absorb_out_kernel(const float* __restrict__ ysum, const __nv_bfloat16* __restrict__ Wv,
                  const __nv_bfloat16* __restrict__ bv, float* __restrict__ out, int B, int n_q_heads, int g,
                  int m, int D, int d_in) {
  __shared__ float red[8][kOutRows][kOutPairs];
  const int kv = blockIdx.x, jt = blockIdx.y, first = blockIdx.z * kOutPairs;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_pairs = B * g;
  const int row0 = kv * 128 + jt * kOutRows;        // flat dim of this block's first output feature
  if (row0 < m) {
    // stored dims (m is a multiple of the block's 16 features): read back as they are
    for (int idx = tid; idx < kOutPairs * kOutRows; idx += 256) {
      const int k = idx / kOutRows, j = jt * kOutRows + idx % kOutRows;
      const int pr = first + k;
      if (pr >= n_pairs) continue;
      const int b = pr / g, h = kv * g + (pr - b * g);
      out[((size_t)b * n_q_heads + h) * 128 + j] = ysum[((size_t)b * n_q_heads + h) * d_in + D + kv * 128 + j];
    }
    return;
  }
  const float* yrow[kOutPairs];
#pragma unroll
  for (int k = 0; k < kOutPairs; ++k) {
    const int pr = min(first + k, n_pairs - 1);       // (pairs past the end repeat the last one; not stored)
    const int b = pr / g, h = kv * g + (pr - b * g);
    yrow[k] = ysum + ((size_t)b * n_q_heads + h) * d_in;
  }
  const __nv_bfloat16* w = Wv + (size_t)(row0 - m) * d_in;
  float acc[kOutRows][kOutPairs];
#pragma unroll
  for (int r = 0; r < kOutRows; ++r)
#pragma unroll
    for (int k = 0; k < kOutPairs; ++k) acc[r][k] = 0.f;
  // warp w takes columns [w * 32 * 4, ...) in steps of 8 warps x 32 lanes x 4 columns
  for (int i = (warp * 32 + lane) * 4; i < d_in; i += 8 * 32 * 4) {
    float yy[kOutPairs][4];
#pragma unroll
    for (int k = 0; k < kOutPairs; ++k) {
      const float4 v = *reinterpret_cast<const float4*>(yrow[k] + i);
      yy[k][0] = v.x; yy[k][1] = v.y; yy[k][2] = v.z; yy[k][3] = v.w;
    }
#pragma unroll
    for (int r = 0; r < kOutRows; ++r) {
      const uint2 raw = *reinterpret_cast<const uint2*>(w + (size_t)r * d_in + i);
      const float wv[4] = {__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u),
                           __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u)};
#pragma unroll
      for (int k = 0; k < kOutPairs; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[r][k] = fmaf(wv[e], yy[k][e], acc[r][k]);
    }
  }
#pragma unroll
  for (int r = 0; r < kOutRows; ++r)
#pragma unroll
    for (int k = 0; k < kOutPairs; ++k) {
      const float tot = warp_sum(acc[r][k]);
      if (lane == 0) red[warp][r][k] = tot;
    }
  __syncthreads();
  if (tid < kOutRows * kOutPairs) {
    const int r = tid / kOutPairs, k = tid % kOutPairs;
    const int pr = first + k;
    if (pr < n_pairs) {
      float res = 0.f;
#pragma unroll
      for (int ww = 0; ww < 8; ++ww) res += red[ww][r][k];
      const int b = pr / g, h = kv * g + (pr - b * g);
      const int j = jt * kOutRows + r;
      if (bv != nullptr) res += __bfloat162float(bv[row0 - m + r]);
      out[((size_t)b * n_q_heads + h) * 128 + j] = res;
    }
  }
}

// out[b][h][:] holds the normalised result over the predicted tokens, ml[b][h] its (max, sum); parts hold the
// partial over the sink / window tokens at index 0.  Combine the two by log-sum-exp.
// bk_shift (may be null): the K predictor's bias, which the absorbed queries leave out; it shifts the scores of a
// predicted head's predicted tokens by q . b_k against the sink / window tokens' true keys.
__global__ void __launch_bounds__(128)
absorb_combine_kernel(float* __restrict__ out, const float2* __restrict__ ml, Partials parts, int n_q_heads,
                      const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ bk_shift, int g, int m,
                      float scale_log2e) {
  const int h = blockIdx.x, b = blockIdx.y, j = threadIdx.x;
  const size_t bh = (size_t)b * n_q_heads + h;
  float2 mid = ml[bh];
  const int flat = (h / g) * 128 + j;              // this thread's flat dim of the head
  if (bk_shift != nullptr && (h / g) * 128 + 127 >= m) {
    __shared__ float s_dot[4];
    float d = flat >= m ? __bfloat162float(q[bh * 128 + j]) * __bfloat162float(bk_shift[flat - m]) : 0.f;
    d = warp_sum(d);
    if ((j & 31) == 0) s_dot[j >> 5] = d;
    __syncthreads();
    mid.x += ((s_dot[0] + s_dot[1]) + (s_dot[2] + s_dot[3])) * scale_log2e;
  }
  const float2 side = parts.ml[bh * parts.max_parts];
  const float M = fmaxf(mid.x, side.x);
  if (M == -INFINITY) return;      // (an unusable sequence: zeros were written already)
  const float w_mid = mid.y > 0.f ? exp2f(mid.x - M) * mid.y : 0.f;      // weight of the normalised mid result
  const float w_side = exp2f(side.x - M);
  const float denom = w_mid + w_side * side.y;
  const float o_side = parts.o[bh * parts.max_parts * 128 + j];
  out[bh * 128 + j] = denom > 0.f ? (w_mid * out[bh * 128 + j] + w_side * o_side) / denom : 0.f;
}

int round_up(int v, int a) { return (v + a - 1) / a * a; }

}  // namespace

bool absorbed_supported(int dtype, int head_dim, int n_q_heads, int n_kv_heads, int m, int page_tokens) {
  if (dtype != ECHOKV_BF16 || head_dim != 128) return false;
  if (n_q_heads != 16 && n_q_heads != 32 && n_q_heads != 64) return false;   // 2 H_q accumulator columns
  if (n_q_heads / n_kv_heads > kMaxGroup) return false;
  if (m < 0 || m % 64 != 0 || m >= n_kv_heads * head_dim) return false;
  return page_tokens == 16 || page_tokens == 32 || page_tokens == 64 || page_tokens == 128;
}

void absorbed_layout(int max_batch, int n_q_heads, int d_in, int capacity_tokens, AbsorbLayout* out) {
  auto align = [](uint64_t v) { return (v + 255) / 256 * 256; };
  out->nh2 = 2 * n_q_heads;
  out->l_cap = round_up(capacity_tokens, kAbsorbTokAlign);
  uint64_t off = 0;
  out->off_q2 = off; off = align(off + (uint64_t)max_batch * out->nh2 * d_in * 2);
  out->off_s = off; off = align(off + (uint64_t)max_batch * n_q_heads * out->l_cap * 4);
  out->off_p2 = off; off = align(off + (uint64_t)max_batch * out->nh2 * out->l_cap * 2);
  out->off_ml = off; off = align(off + (uint64_t)max_batch * n_q_heads * 8);
  out->off_ml_range = off; off = align(off + (uint64_t)max_batch * n_q_heads * kAbsorbMaxRanges * 8);
  out->off_y = off; off = align(off + (uint64_t)max_batch * kAbsorbMaxRanges * n_q_heads * d_in * 4);
  out->off_ysum = off; off = align(off + (uint64_t)max_batch * n_q_heads * d_in * 4);
  out->total = off;
}

cudaError_t absorbed_encode_maps(AbsorbMaps* maps, unsigned char* ws, const AbsorbLayout& lay, int max_batch, int d_in) {
  cudaError_t e = encode_chunked_3d_map(&maps->q2, ws + lay.off_q2, (uint64_t)max_batch * lay.nh2, d_in, lay.nh2, 2);
  if (e != cudaSuccess) return e;
  e = encode_pool_box_map(&maps->p2, ws + lay.off_p2, lay.l_cap, (uint64_t)max_batch * lay.nh2, lay.nh2);
  if (e != cudaSuccess) return e;
  maps->ready = true;
  return cudaSuccess;
}

cudaError_t launch_absorbed(const AttnArgs& a, const AbsorbArgs& r, const AbsorbMaps& maps, const TcLayerMaps& anchor,
                            const TcLayerMaps& layer, float* out, int sm_count, cudaStream_t stream,
                            cudaEvent_t* ev) {
  if (!maps.ready || !anchor.pools_ready) return cudaErrorInvalidValue;
  if (r.m > 0 && !layer.pools_ready) return cudaErrorInvalidValue;
  if (a.batch > kMaxBatchPerLaunch) return cudaErrorInvalidValue;
  const int g = a.n_q_heads / a.n_kv_heads;
  const int d_in = r.D + r.m;
  const int m_heads = r.m_heads >= 0 ? r.m_heads : r.m / 128 * 128;
  const int n_ret = m_heads / 128;       // whole retained heads: scored from the pool when the keys are rotated
  const AbsorbLayout& lay = r.lay;
  __nv_bfloat16* q2 = reinterpret_cast<__nv_bfloat16*>(r.ws + lay.off_q2);
  float* S = reinterpret_cast<float*>(r.ws + lay.off_s);
  __nv_bfloat16* p2 = reinterpret_cast<__nv_bfloat16*>(r.ws + lay.off_p2);
  float2* ml = reinterpret_cast<float2*>(r.ws + lay.off_ml);
  float2* ml_range = reinterpret_cast<float2*>(r.ws + lay.off_ml_range);
  float* y = reinterpret_cast<float*>(r.ws + lay.off_y);
  float* ysum = reinterpret_cast<float*>(r.ws + lay.off_ysum);
  cudaError_t e;

  const bool rotated = a.rope.cs != nullptr;
  if (rotated && !r.save_k && !layer.weights_ready) return cudaErrorInvalidValue;
  // K side: features [anchor dims ; retained dims] and Wk^T q -- or, where the layer keeps its keys whole, the
  // layer's own D key dims with every query placed at its head's dims
  const int k_m = r.save_k ? r.D : r.m, k_anchor_dims = r.save_k ? 0 : r.D;

  // 1. absorbed queries
  if (!rotated) {
    dim3 grid((d_in + kQCols - 1) / kQCols, a.n_kv_heads, (a.batch * g + kQGroup - 1) / kQGroup);
    if ((e = cudaFuncSetAttribute(absorb_query_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)kQuerySmemBytes)) != cudaSuccess)
      return e;
    // several blocks per SM: ask for the largest shared-memory carve-out (the default sizes it for one block)
    if ((e = cudaFuncSetAttribute(absorb_query_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                  cudaSharedmemCarveoutMaxShared)) != cudaSuccess)
      return e;
    absorb_query_kernel<<<grid, 256, kQuerySmemBytes, stream>>>(reinterpret_cast<const __nv_bfloat16*>(a.q),
                                                  reinterpret_cast<const __nv_bfloat16*>(r.Wk), q2, a.batch,
                                                  a.n_q_heads, g, k_m, k_anchor_dims, d_in, a.scale_log2e);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }

  StreamParams p;
  p.slots = a.slots;
  p.lens = a.lens;
  p.table = a.geom.table;
  p.max_batch = a.geom.max_batch;
  p.max_pages_per_seq = a.geom.max_pages_per_seq;
  p.page_tokens = a.geom.page_tokens;
  p.n_pages = a.geom.n_pages;
  p.status = a.status;
  p.b0 = 0;
  p.nb = a.batch;
  p.n_q_heads = a.n_q_heads;
  p.nh2 = lay.nh2;
  p.kc_anchor = r.D / kChunk;
  p.kc_total = d_in / kChunk;
  p.run_pages = a.geom.page_tokens < kRunTokens ? kRunTokens / a.geom.page_tokens : 1;
  p.l_cap = lay.l_cap;
  p.n_sink = r.n_sink;
  p.n_window = r.n_window;
  p.s_out = S;
  p.y_out = y;
  p.d_in = d_in;
  // with m == 0 the local maps are never used; pass the anchor's so the parameters stay valid
  const TcLayerMaps& loc = r.m > 0 ? layer : anchor;
  const int capacity = r.capacity_tokens;

  // 2. scores
  if (rotated) {
    // keys rotated by position: predicted heads on the tensor cores (Eq. 3, rotation, q . k), stored heads from
    // the layer's pool; both write the score rows the softmax below reads
    ReconArgs ra;
    ra.k_anchor = nullptr; ra.v_anchor = nullptr; ra.k_local = r.k_local; ra.v_local = r.v_local;
    ra.Wk = r.Wk_x != nullptr ? r.Wk_x : r.Wk; ra.Wv = r.Wv;
    ra.bk = r.bk != nullptr ? (r.Wk_x != nullptr ? r.bk_x : r.bk) : nullptr;
    ra.D = r.D; ra.m = r.m; ra.m_heads = m_heads;
    ra.part_tokens = 0;
    ra.capacity_tokens = capacity;
    ra.n_sink = r.n_sink; ra.n_window = r.n_window;
    if (ev) cudaEventRecord(ev[0], stream);
    if (r.save_k) {
      if (r.k_stored == nullptr) return cudaErrorInvalidValue;
      if ((e = launch_key_scores_stored(a, *r.k_stored, *r.k_stored_run, a.n_kv_heads, S, lay.l_cap, r.n_sink,
                                        r.n_window, sm_count, stream)) != cudaSuccess)
        return e;
    } else {
      if ((e = launch_recon_pair_key_scores(a, ra, anchor, layer, S, lay.l_cap, sm_count, stream)) != cudaSuccess) return e;
      if (n_ret > 0) {
        if (r.k_stored == nullptr) return cudaErrorInvalidValue;
        if ((e = launch_key_scores_stored(a, *r.k_stored, *r.k_stored_run, n_ret, S, lay.l_cap, r.n_sink, r.n_window,
                                          sm_count, stream)) != cudaSuccess)
          return e;
      }
    }
    if (ev) cudaEventRecord(ev[1], stream);
  } else {
    const TcLayerMaps& k_loc = r.save_k ? layer : loc;
    if (r.save_k) {         // the K pass streams the layer's own keys only
      p.kc_anchor = 0;
      p.kc_total = r.D / kChunk;
    }
    p.stage_bytes = 2u * (kScoreXBytes + (uint32_t)lay.nh2 * kRowBytes);
    p.n_stages = (int)(kSmemBudget / p.stage_bytes);
    if (p.n_stages > kMaxStages) p.n_stages = kMaxStages;
    p.idesc = make_idesc(lay.nh2, false);
    p.range_tokens = 0; p.n_slices = 0;
    const size_t smem = 1024 + (size_t)p.n_stages * p.stage_bytes + sizeof(StreamSmemTail);
    if ((e = cudaFuncSetAttribute(absorb_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
        cudaSuccess)
      return e;
    const long long max_items = (long long)a.batch * ((capacity + kScoreTokens - 1) / kScoreTokens);
    const int grid = (int)(max_items < sm_count ? max_items : sm_count);
    if (ev) cudaEventRecord(ev[0], stream);
    absorb_scores_kernel<<<grid, kThreads, smem, stream>>>(anchor.k_grp_page, k_loc.k_grp_page, anchor.k_grp_64,
                                                           k_loc.k_grp_64, anchor.k_grp_128, k_loc.k_grp_128,
                                                           maps.q2, p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (ev) cudaEventRecord(ev[1], stream);
    p.kc_anchor = r.D / kChunk;      // (the V pass streams [anchor dims ; retained dims] in any case)
    p.kc_total = d_in / kChunk;
  }

  // the V pass splits every sequence into token ranges; the softmax works range by range as well
  int range_tokens;
  {
    p.n_slices = (p.kc_total + 3) / 4;
    // about ten items per CTA so that the persistent grid ends evenly, but ranges of >= 1024 tokens so that
    // the partial results stay small next to what a range reads
    int ranges = (10 * sm_count + p.n_slices * a.batch - 1) / (p.n_slices * a.batch);
    if (ranges > kAbsorbMaxRanges) ranges = kAbsorbMaxRanges;
    if (ranges < 1) ranges = 1;
    range_tokens = round_up((capacity + ranges - 1) / ranges, kPvTokens);
    if (range_tokens < 1024) range_tokens = 1024;
  }

  // 3. per range: maximum, sum, probabilities
  {
    dim3 grid(a.n_q_heads, a.batch, (capacity + range_tokens - 1) / range_tokens);
    absorb_softmax_kernel<<<grid, 256, 0, stream>>>(S, p2, ml_range, a.slots, a.lens, a.geom.max_batch, capacity,
                                                    a.n_q_heads, lay.l_cap, range_tokens);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }

  // 4. probability-weighted inputs
  {
    p.range_tokens = range_tokens;
    p.stage_bytes = kPvVBytes + (uint32_t)lay.nh2 * kRowBytes;
    p.n_stages = (int)(kSmemBudget / p.stage_bytes);
    if (p.n_stages > kMaxStages) p.n_stages = kMaxStages;
    p.idesc = make_idesc(lay.nh2, true);
    const size_t smem = 1024 + (size_t)p.n_stages * p.stage_bytes + sizeof(StreamSmemTail);
    if ((e = cudaFuncSetAttribute(absorb_pv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) !=
        cudaSuccess)
      return e;
    const long long max_items = (long long)a.batch * ((capacity + range_tokens - 1) / range_tokens) * p.n_slices;
    const int grid = (int)(max_items < sm_count ? max_items : sm_count);
    if (ev) cudaEventRecord(ev[2], stream);
    absorb_pv_kernel<<<grid, kThreads, smem, stream>>>(anchor.v_grp_page, loc.v_grp_page, anchor.v_grp_64, loc.v_grp_64,
                                                       maps.p2, p);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (ev) cudaEventRecord(ev[3], stream);
  }

  // 5. sum the ranges, normalise, project
  {
    dim3 grid1((d_in / 4 + 255) / 256, a.n_q_heads, a.batch);
    absorb_ysum_kernel<<<grid1, 256, 0, stream>>>(y, ml_range, ml, ysum, a.slots, a.lens, a.geom.max_batch, capacity,
                                                  a.n_q_heads, d_in, range_tokens);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    dim3 grid2(a.n_kv_heads, 128 / kOutRows, (a.batch * g + kOutPairs - 1) / kOutPairs);
    absorb_out_kernel<<<grid2, 256, 0, stream>>>(ysum, reinterpret_cast<const __nv_bfloat16*>(r.Wv),
                                                 reinterpret_cast<const __nv_bfloat16*>(r.bv), out, a.batch,
                                                 a.n_q_heads, g, r.m, r.D, d_in);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  // 6. sink and recent-window tokens (Section 4.1): attended at full precision by the side kernel, then
  //    combined with the result over the predicted tokens
  if (r.n_sink > 0 || r.n_window > 0) {
    SideArgs side;
    side.k_side = r.k_side; side.v_side = r.v_side;
    side.n_sink = r.n_sink; side.n_window = r.n_window; side.d_drop = r.D - r.m;
    SidePool pool;
    pool.k_pool = r.k_local; pool.v_pool = r.v_local; pool.width = r.m; pool.part = 0;
    pool.k_width = r.save_k ? r.D : 0;
    if ((e = launch_attn_side(a, side, 0, 1, stream, pool)) != cudaSuccess) return e;
    dim3 grid(a.n_q_heads, a.batch);
    absorb_combine_kernel<<<grid, 128, 0, stream>>>(out, ml, a.parts, a.n_q_heads,
                                                    reinterpret_cast<const __nv_bfloat16*>(a.q),
                                                    reinterpret_cast<const __nv_bfloat16*>(r.bk_shift), g, r.m,
                                                    a.scale_log2e);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace echokv
