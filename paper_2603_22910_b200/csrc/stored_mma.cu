// Attention over heads that are stored in the cache (anchor layers, the retained heads of a
// compressed layer, the uncompressed mode): Eq. 7 straight on the paged bf16 cache.
//
// The work is a pure HBM stream (512 bytes of K and V per token and KV head, a few hundred
// FLOP), so the kernel is built around keeping many bytes in flight:
//
//   persistent grid, two CTAs per SM, 160 threads: warp 0 issues TMA, warps 1..4 consume
//   work item  = (sequence, range of item_tokens tokens, KV head), heads fastest so that the
//                CTAs running together read the same DRAM rows
//   stage      = 64 tokens of one head: K and V as two 64-feature boxes each (page-sized TMA
//                boxes taken through the block table, 128-byte swizzle), 32 KiB, 3 deep
//   consumer   : every warp takes 16 tokens of every stage, with its own running (max, sum, O), so
//                that each warp sees every phase of every stage barrier.  S = Q K^T and O += P V run
//                as mma.sync m16n8k16 with the query heads of the group on the M rows; the group has
//                at most 8 query heads, so M rows 8..15 carry the low-order bf16 half of P
//                (P = P_hi + P_lo), which keeps the probabilities at ~16 mantissa bits for free.
//                Online softmax in fp32 registers, base-2 exponent units.
//   item end   : the four warps' (max, sum, O) are combined in shared memory into one split-K
//                partial; the merge kernel combines the items of a sequence.
//
// item_tokens is chosen inside the kernel from the lengths actually present (all CTAs compute
// the same value) and published for the merge kernel.  Every wait is bounded.
#include "stored_mma.h"

#include "ptx_sm100.cuh"

namespace echokv {

namespace {

constexpr int kStages = 3;                           // stage barriers in shared memory (stages in use: StoredStages)
constexpr int kFineRowPairs = 72;                    // (cos, sin) pairs per row of the in-CTA offset table: 64 + 8 of
                                                     // padding, so that two rows fill the 32 banks exactly
// Stages of 32 KiB per CTA.  The rotating variant also keeps a 9 KiB table; with many query heads per KV
// head (a large merge area) it runs on two stages so that two CTAs still fit an SM.
template <int G, bool ROPE>
struct StoredStages { static constexpr int value = (ROPE && G >= 4) ? 2 : 3; };
constexpr int kStageTokens = 64;
constexpr int kBlockBytes = kStageTokens * 128;      // 64 token rows x 64 features (128 bytes)
constexpr int kStageBytes = 4 * kBlockBytes;         // K (both 64-feature halves of the head), then V
// Inside the K (or V) half of a stage the rows sit as 1 KiB swizzle atoms (8 rows x 64 features) in the order
// (8-row group, feature half): one TMA box brings both halves of a page's rows (the pools are described to TMA as
// [group][chunk][row of the group][64]).  Byte offset of 16-byte piece `piece` (0..15 over the head's 128 features)
// of token row `tok` of the stage:
__device__ __forceinline__ uint32_t stage_off(int tok, int piece) {
  return (uint32_t)((tok >> 3) * 2048 + (piece >> 3) * 1024 + (tok & 7) * 128 + (((piece & 7) ^ (tok & 7)) << 4));
}
constexpr int kConsumers = 4;
constexpr int kWarpTokens = kStageTokens / kConsumers;   // every consumer warp takes 16 tokens of each stage
constexpr int kThreads = 32 * (1 + kConsumers);
constexpr int kMinItemTokens = 256;
constexpr int kMaxItemTokens = 16384;
constexpr int kItemsPerCta = 6;                      // target number of work items per CTA

struct StoredParams {
  const __nv_bfloat16* q;
  const int32_t* slots;
  const int32_t* lens;
  const int32_t* table;
  int max_batch, max_pages_per_seq, page_tokens;
  long long n_pages;
  float2* part_ml;
  float* part_o;
  int max_parts;
  int32_t* status;
  int32_t* item_tokens_out;   // where this launch publishes its item_tokens
  int b0, nb;                 // batch entries [b0, b0 + nb) are handled by this launch
  int n_q_heads, n_heads;     // query heads in all; stored KV heads attended (0 .. n_heads - 1)
  int rows_per_box;           // token rows per TMA box: min(page_tokens, 64)
  float scale_log2e;
  RopeTable rope;             // read by the ROPE instantiations only
};

template <int G>
struct StoredSmemTail {
  float mo[kConsumers][G][128];
  float mm[kConsumers][8];
  float ml[kConsumers][8];
  int cum_items[kStoredMaxBatchPerLaunch + 1];
  unsigned long long full_bar[kStages];
  unsigned long long empty_bar[kStages];
  uint32_t box_ok[kStages];
  unsigned long long total_tokens;
  int item_tokens;
  int abort_flag;
};

__device__ __forceinline__ void consumers_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// Barrier over the four consumer warps that also ANDs a flag (see the bounded waits).
__device__ __forceinline__ bool consumers_all(bool ok) {
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

struct Item {
  int b;          // index inside this launch's batch slice
  int chunk;      // which item_tokens-sized range of the sequence
  int kvh;
};

template <int G>
__device__ __forceinline__ Item decode_item(const StoredSmemTail<G>& t, int item, int n_heads, int nb) {
  int lo = 0, hi = nb;   // largest b with cum_items[b] <= item
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (t.cum_items[mid] <= item) lo = mid; else hi = mid;
  }
  Item it;
  it.b = lo;
  const int local = item - t.cum_items[lo];
  it.chunk = local / n_heads;
  it.kvh = local - it.chunk * n_heads;
  return it;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// two packed bf16 -> fp32
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }
// (x0, x1) as a packed bf16 pair plus the packed pair of what the rounding dropped
__device__ __forceinline__ void split_bf16(float x0, float x1, uint32_t& head, uint32_t& rest) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  head = *reinterpret_cast<const uint32_t*>(&h);
  rest = pack_bf16(x0 - __low2float(h), x1 - __high2float(h));
}

// ROPE: every key row is rotated to its position before q . k (Section 3.2: the cache holds keys prior to
// the rotary embedding).  The rotated rows are formed in fp32 from the fragments and fed to the tensor
// cores as bf16 head + remainder, so the rotation costs no precision.
template <int G, bool ROPE>
__global__ void __launch_bounds__(kThreads, 2)
attn_stored_mma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       const __grid_constant__ CUtensorMap tm_k_run, const __grid_constant__ CUtensorMap tm_v_run,
                       const StoredParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  constexpr int NS = StoredStages<G, ROPE>::value;
  StoredSmemTail<G>& t = *reinterpret_cast<StoredSmemTail<G>*>(smem + NS * kStageBytes);
  // ROPE: (cos, sin)(r * w_j) for the 16 offsets r inside a warp's token slice, rows padded (see kFineRowPairs)
  float2* fine = reinterpret_cast<float2*>(smem + NS * kStageBytes + ((sizeof(StoredSmemTail<G>) + 15) / 16) * 16);
  if constexpr (ROPE) {
    for (int i = threadIdx.x; i < kRopeFineRows * 64; i += kThreads)
      fine[(i >> 6) * kFineRowPairs + (i & 63)] = p.rope.fine[i];
  }
  const uint32_t stage_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &t.abort_flag;
  const int capacity = p.max_pages_per_seq * p.page_tokens;

  // ---- set-up: item size from the lengths present, items per sequence, barriers -----------------
  if (tid == 0) {
    t.total_tokens = 0ull;
    t.abort_flag = 0;
    t.cum_items[0] = 0;
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&t.full_bar[s]), 1);
      mbar_init(smem_u32(&t.empty_bar[s]), kConsumers);
    }
    mbar_fence_init();
  }
  __syncthreads();
  {
    unsigned long long mine = 0ull;
    for (int i = tid; i < p.nb; i += kThreads) {
      const int b = p.b0 + i;
      const int slot = p.slots ? p.slots[b] : b;
      const int len = p.lens[b];
      if (slot < 0 || slot >= p.max_batch) {
        if (blockIdx.x == 0) report(p.status, ECHOKV_EBADPAGE);
      } else if (len < 1 || len > capacity) {
        if (blockIdx.x == 0) report(p.status, ECHOKV_EBADLENGTH);
      } else {
        mine += (unsigned long long)len;
      }
    }
    if (mine) atomicAdd(&t.total_tokens, mine);
  }
  __syncthreads();
  if (tid == 0) {
    // about kItemsPerCta items per CTA, in whole multiples of 256 tokens (64 per consumer warp)
    const unsigned long long want = (unsigned long long)kItemsPerCta * gridDim.x;
    unsigned long long per_item = (t.total_tokens * (unsigned long long)p.n_heads + want - 1) / want;
    per_item = (per_item + kMinItemTokens - 1) / kMinItemTokens * kMinItemTokens;
    if (per_item < kMinItemTokens) per_item = kMinItemTokens;
    if (per_item > kMaxItemTokens) per_item = kMaxItemTokens;
    t.item_tokens = (int)per_item;
    if (blockIdx.x == 0) *p.item_tokens_out = (int)per_item;
  }
  __syncthreads();
  const int item_tokens = t.item_tokens;
  for (int i = tid; i < p.nb; i += kThreads) {
    const int b = p.b0 + i;
    const int slot = p.slots ? p.slots[b] : b;
    const int len = p.lens[b];
    const bool ok = slot >= 0 && slot < p.max_batch && len >= 1 && len <= capacity;
    t.cum_items[i + 1] = ok ? ((len + item_tokens - 1) / item_tokens) * p.n_heads : 0;
  }
  __syncthreads();
  if (warp == 0) {
    // inclusive scan of cum_items[1 .. nb], 32 entries at a time
    int carry = 0;
    for (int base = 0; base < p.nb; base += 32) {
      const int i = base + lane;
      int v = i < p.nb ? t.cum_items[i + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
      }
      if (i < p.nb) t.cum_items[i + 1] = v + carry;
      carry += __shfl_sync(0xffffffffu, v, 31);
    }
  }
  __syncthreads();
  const int n_items = t.cum_items[p.nb];
  const int rpb = p.rows_per_box;
  const int n_boxes = (kStageTokens / rpb) * 4;

  if (warp == 0) {
    // =============================== TMA producer ===============================================
    uint32_t it = 0;
    uint32_t issued[NS];
#pragma unroll
    for (int s = 0; s < NS; ++s) issued[s] = 0;
    bool alive = true;
    const int sub = lane >> 2, kind = lane & 3;    // box row group inside the stage; K lo, K hi, V lo, V hi
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Item w = decode_item<G>(t, item, p.n_heads, p.nb);
      const int b = p.b0 + w.b;
      const int slot = p.slots ? p.slots[b] : b;
      const int len = p.lens[b];
      const int t_begin = w.chunk * item_tokens;
      const int t_end = min(len, t_begin + item_tokens);
      const int n_iter = (t_end - t_begin + kStageTokens - 1) / kStageTokens;
      const int32_t* table = p.table + (size_t)slot * p.max_pages_per_seq;
      // block-table entry of this lane's box of stage j (requested one stage ahead of its use)
      auto load_page = [&](int j) {
        const int tb = t_begin + j * kStageTokens + sub * rpb;
        return (lane < n_boxes && tb < t_end) ? table[tb / p.page_tokens] : -1;
      };
      int page_next = load_page(0);
      for (int j = 0; j < n_iter; ++j, ++it) {
        const int page = page_next;
        if (j + 1 < n_iter) page_next = load_page(j + 1);
        const uint32_t s = it % NS;
        const uint32_t ph = (it / NS) & 1u;
        bool ok = true;
        if (lane == 0) ok = mbar_wait(smem_u32(&t.empty_bar[s]), ph ^ 1u, abort_flag, p.status);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) { alive = false; break; }
        const int tb = t_begin + j * kStageTokens + sub * rpb;      // first token of this lane's box
        long long row = -1;
        if (lane < n_boxes && tb < t_end) {
          if (page < 0 || page >= p.n_pages) {
            report(p.status, ECHOKV_EBADPAGE);
          } else {
            row = (long long)page * p.page_tokens + tb % p.page_tokens;
          }
        }
        const uint32_t ok_mask = __ballot_sync(0xffffffffu, row >= 0);
        // all boxes of the stage cached and consecutive in the pool: one 64-row copy per kind instead of one
        // per page (lanes 0..3 hold the first page's row for the four kinds)
        const long long row0 = __shfl_sync(0xffffffffu, row, kind);
        const bool run = n_boxes > 4 && __all_sync(0xffffffffu, lane >= n_boxes || (row >= 0 && row == row0 + sub * rpb));
        const uint32_t full = smem_u32(&t.full_bar[s]);
        if (lane == 0) {
          t.box_ok[s] = ok_mask;
          mbar_arrive_expect_tx(full, __popc(ok_mask) * (uint32_t)rpb * 128u);
        }
        __syncwarp();
        // (lanes of kinds 0 and 2 copy: one box holds both feature halves, K or V)
        if (run) {
          if (lane < 4 && (kind & 1) == 0)
            tma_load_4d(stage_base + s * kStageBytes + kind * kBlockBytes, kind < 2 ? &tm_k_run : &tm_v_run, 0, 0,
                        w.kvh * 2, (int)(row >> 3), full);
        } else if (row >= 0 && (kind & 1) == 0) {
          tma_load_4d(stage_base + s * kStageBytes + kind * kBlockBytes + sub * rpb * 256,
                      kind < 2 ? &tm_k : &tm_v, 0, 0, w.kvh * 2, (int)(row >> 3), full);
        }
        issued[s] = it + 1;
      }
    }
    if (!alive && lane == 0) {
      // let every copy this warp started land before the CTA leaves
#pragma unroll
      for (int s = 0; s < NS; ++s)
        if (issued[s] != 0) mbar_drain(smem_u32(&t.full_bar[s]), ((issued[s] - 1) / NS) & 1u);
    }
  } else {
    // =============================== consumers (4 warps) ========================================
    const int cw = warp - 1;
    const int row = lane >> 2;                // query head of the group held in c0 / c1
    const int qd = (lane & 3) * 2;            // first of this thread's two columns inside an 8-wide tile
    const int ct = tid - 32;                  // 0..127: output feature at the item-end merge
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Item w = decode_item<G>(t, item, p.n_heads, p.nb);
      const int b = p.b0 + w.b;
      const int len = p.lens[b];
      const int t_begin = w.chunk * item_tokens;
      const int t_end = min(len, t_begin + item_tokens);
      const int n_iter = (t_end - t_begin + kStageTokens - 1) / kStageTokens;

      // A fragments of Q: rows 0..G-1 are the group's query heads, the rest is zero
      uint32_t qa0[8], qa2[8];
      {
        const __nv_bfloat16* qrow = p.q + ((size_t)b * p.n_q_heads + (size_t)w.kvh * G + row) * 128 + qd;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          qa0[ks] = row < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16) : 0u;
          qa2[ks] = row < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8) : 0u;
        }
      }
      float m_run = -INFINITY, l_run = 0.f;
      float o[16][4];
#pragma unroll
      for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;

      // ROPE: the angle of token 16 u + r is the sum of a coarse angle (row u of the coarse table, fetched a
      // stage ahead of its use) and a fine one (row r of the table in shared memory).  base[2 ks + h] holds the
      // coarse (cos, sin) of this thread's frequency indices 16 ks + 8 h + qd and + 1, which pair feature jj of
      // the first 64-feature block with feature jj + 64.
      float4 base[ROPE ? 8 : 1];
      auto load_base = [&](int stage_t0) {
        if constexpr (ROPE) {
          const int u = min(stage_t0 / kRopeFineRows + cw, p.rope.stride / kRopeFineRows - 1);
          const float4* src = reinterpret_cast<const float4*>(p.rope.coarse + (size_t)u * 64 + qd);
#pragma unroll
          for (int k = 0; k < 8; ++k) base[k] = __ldg(src + k * 4);
        }
      };
      load_base(t_begin);

      for (int j = 0; j < n_iter; ++j, ++it) {
        const uint32_t s = it % NS;
        const uint32_t ph = (it / NS) & 1u;
        const bool got = mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
        const uint32_t sb = stage_base + s * kStageBytes;
        const int t0 = t_begin + j * kStageTokens;
        const uint32_t ok_mask = t.box_ok[s];
        // bit i: token i of this warp's 16-token slice of the stage holds a cached token
        uint32_t vmask;
        {
          const int n_tok = min(kStageTokens, t_end - t0);
          const unsigned long long in_len = n_tok >= 64 ? ~0ull : ((1ull << n_tok) - 1ull);
          unsigned long long in_box = 0ull;
          const unsigned long long box_bits = rpb >= 64 ? ~0ull : ((1ull << rpb) - 1ull);
          for (int g = 0; g < kStageTokens / rpb; ++g)
            if ((ok_mask >> (g * 4)) & 1u) in_box |= box_bits << (g * rpb);
          vmask = (uint32_t)((in_len & in_box) >> (cw * kWarpTokens)) & 0xffffu;
        }
        if (vmask != 0u) {
          const bool all_valid = vmask == 0xffffu;
          const int tok_k = cw * kWarpTokens + (lane >> 4) * 8 + (lane & 7);          // K rows: ldmatrix
          const int tok_v = cw * kWarpTokens + ((lane >> 3) & 1) * 8 + (lane & 7);    // V rows: ldmatrix.trans
          if (!all_valid) {
            // rows without a cached token may hold anything (never written, or a skipped page):
            // zero them in V so that 0 * V stays 0; their scores are masked below
            for (int idx = lane; idx < kWarpTokens * 16; idx += 32) {
              const int r = idx >> 4, piece = idx & 15;
              if (!((vmask >> r) & 1u)) {
                // (every piece of the row is zeroed, so the swizzle does not matter: any order of its 16 pieces)
                const uint32_t a = sb + 2 * kBlockBytes + stage_off(cw * kWarpTokens + r, piece);
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0u) : "memory");
              }
            }
            __syncwarp();
          }

          // ---- S = Q K^T: two token tiles of 8, contraction over 128 features ----
          float sc[2][4];
#pragma unroll
          for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[nt][e] = 0.f;
          if constexpr (ROPE) {
            // register i of step ks: token tile i >> 1 (slice offsets lane / 4 and lane / 4 + 8), frequency
            // indices 16 ks + 8 (i & 1) + qd and + 1
            const float4* fine_a = reinterpret_cast<const float4*>(fine + (lane >> 2) * kFineRowPairs + qd);
            const float4* fine_b = reinterpret_cast<const float4*>(fine + ((lane >> 2) + 8) * kFineRowPairs + qd);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const int c0 = ks * 2 + ((lane >> 3) & 1);
              uint32_t a[4], b[4];
              ldsm_x4(sb + stage_off(tok_k, c0), a[0], a[1], a[2], a[3]);
              ldsm_x4(sb + stage_off(tok_k, 8 + c0), b[0], b[1], b[2], b[3]);
              uint32_t lo_h[4], lo_r[4], hi_h[4], hi_r[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float4 bw = base[ks * 2 + (i & 1)];
                const float4 fw = ((i >> 1) ? fine_b : fine_a)[ks * 8 + (i & 1) * 4];
                const float c0w = bw.x * fw.x - bw.y * fw.y, s0w = bw.y * fw.x + bw.x * fw.y;
                const float c1w = bw.z * fw.z - bw.w * fw.w, s1w = bw.w * fw.z + bw.z * fw.w;
                const float a0 = bf16_lo(a[i]), a1 = bf16_hi(a[i]), b0 = bf16_lo(b[i]), b1 = bf16_hi(b[i]);
                split_bf16(a0 * c0w - b0 * s0w, a1 * c1w - b1 * s1w, lo_h[i], lo_r[i]);
                split_bf16(b0 * c0w + a0 * s0w, b1 * c1w + a1 * s1w, hi_h[i], hi_r[i]);
              }
              mma_m16n8k16_bf16(sc[0], qa0[ks], 0u, qa2[ks], 0u, lo_h[0], lo_h[1]);
              mma_m16n8k16_bf16(sc[1], qa0[ks], 0u, qa2[ks], 0u, lo_h[2], lo_h[3]);
              mma_m16n8k16_bf16(sc[0], qa0[ks + 4], 0u, qa2[ks + 4], 0u, hi_h[0], hi_h[1]);
              mma_m16n8k16_bf16(sc[1], qa0[ks + 4], 0u, qa2[ks + 4], 0u, hi_h[2], hi_h[3]);
              mma_m16n8k16_bf16(sc[0], qa0[ks], 0u, qa2[ks], 0u, lo_r[0], lo_r[1]);
              mma_m16n8k16_bf16(sc[1], qa0[ks], 0u, qa2[ks], 0u, lo_r[2], lo_r[3]);
              mma_m16n8k16_bf16(sc[0], qa0[ks + 4], 0u, qa2[ks + 4], 0u, hi_r[0], hi_r[1]);
              mma_m16n8k16_bf16(sc[1], qa0[ks + 4], 0u, qa2[ks + 4], 0u, hi_r[2], hi_r[3]);
            }
            if (j + 1 < n_iter) load_base(t0 + kStageTokens);   // in flight during the rest of this stage
          } else {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const int c0 = (ks & 3) * 2 + ((lane >> 3) & 1);
            uint32_t r0, r1, r2, r3;
            ldsm_x4(sb + stage_off(tok_k, (ks >> 2) * 8 + c0), r0, r1, r2, r3);
            mma_m16n8k16_bf16(sc[0], qa0[ks], 0u, qa2[ks], 0u, r0, r1);
            mma_m16n8k16_bf16(sc[1], qa0[ks], 0u, qa2[ks], 0u, r2, r3);
          }
          }

          // ---- online softmax on row `row` (c0, c1 of both tiles) ----
          float mx = -INFINITY;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              float v = sc[nt][e] * p.scale_log2e;
              if (!all_valid && !((vmask >> (nt * 8 + qd + e)) & 1u)) v = -INFINITY;
              sc[nt][e] = v;
              mx = fmaxf(mx, v);
            }
          }
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          const float m_new = fmaxf(m_run, mx);     // finite: the slice has a valid token
          const float alpha = exp2f(m_run - m_new);
          m_run = m_new;
          uint32_t p_hi[2], p_lo[2];
          float psum = 0.f;
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const float p0 = exp2f(sc[nt][0] - m_new);
            const float p1 = exp2f(sc[nt][1] - m_new);
            psum += p0 + p1;
            const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
            p_hi[nt] = *reinterpret_cast<const uint32_t*>(&h);
            p_lo[nt] = pack_bf16(p0 - __low2float(h), p1 - __high2float(h));
          }
          l_run = l_run * alpha + psum;
          if (alpha != 1.f) {     // (the quad shares alpha, and nothing below is warp-collective per tile)
#pragma unroll
            for (int nt = 0; nt < 16; ++nt)
#pragma unroll
              for (int e = 0; e < 4; ++e) o[nt][e] *= alpha;
          }
          __syncwarp();

          // ---- O += P V: rows 0..7 take P_hi, rows 8..15 take P_lo ----
#pragma unroll
          for (int dp = 0; dp < 8; ++dp) {
            const int chunk = 2 * dp + (lane >> 4);
            uint32_t r0, r1, r2, r3;
            ldsm_x4_trans(sb + 2 * kBlockBytes + stage_off(tok_v, chunk), r0, r1, r2, r3);
            mma_m16n8k16_bf16(o[2 * dp], p_hi[0], p_lo[0], p_hi[1], p_lo[1], r0, r1);
            mma_m16n8k16_bf16(o[2 * dp + 1], p_hi[0], p_lo[0], p_hi[1], p_lo[1], r2, r3);
          }
          if (!all_valid) fence_proxy_async_smem();   // the zeroed rows, before TMA writes there again
        } else if (ROPE && j + 1 < n_iter) {
          load_base(t0 + kStageTokens);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&t.empty_bar[s]));
      }

      // ---- item end: combine the four warps into one partial ----
      if (!consumers_all(alive)) { alive = false; break; }   // (also: previous item's merge area is free)
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
      if (row < G) {
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
          *reinterpret_cast<float2*>(&t.mo[cw][row][nt * 8 + qd]) =
              make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
        if ((lane & 3) == 0) {
          t.mm[cw][row] = m_run;
          t.ml[cw][row] = l_run;
        }
      }
      consumers_sync();
#pragma unroll
      for (int gi = 0; gi < G; ++gi) {
        float M = t.mm[0][gi];
#pragma unroll
        for (int c = 1; c < kConsumers; ++c) M = fmaxf(M, t.mm[c][gi]);
        float L = 0.f, acc = 0.f;
        if (M > -INFINITY) {
#pragma unroll
          for (int c = 0; c < kConsumers; ++c) {
            const float wgt = exp2f(t.mm[c][gi] - M);
            L = fmaf(wgt, t.ml[c][gi], L);
            acc = fmaf(wgt, t.mo[c][gi][ct], acc);
          }
        }
        const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)w.kvh * G + gi) * p.max_parts + w.chunk;
        p.part_o[pidx * 128 + ct] = acc;
        if (ct == 0) p.part_ml[pidx] = make_float2(M, L);
      }
    }
  }
}

template <int G, bool ROPE>
constexpr size_t stored_smem_bytes() {
  return 1024 + (size_t)StoredStages<G, ROPE>::value * kStageBytes + ((sizeof(StoredSmemTail<G>) + 15) / 16) * 16 +
         (ROPE ? (size_t)kRopeFineRows * kFineRowPairs * sizeof(float2) : 0);
}

template <int G, bool ROPE>
cudaError_t launch_g(const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& k_run, const CUtensorMap& v_run,
                     const StoredParams& p, int sm_count, cudaStream_t stream) {
  const size_t smem = stored_smem_bytes<G, ROPE>();
  cudaError_t e = cudaFuncSetAttribute(attn_stored_mma_kernel<G, ROPE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  // as many CTAs as stay resident, but never more than the items there can be
  static int resident = 0;   // per instantiation; the answer depends only on the kernel and the device type
  if (resident == 0) {
    int n = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, attn_stored_mma_kernel<G, ROPE>, kThreads, smem);
    if (e != cudaSuccess) return e;
    resident = n < 1 ? 1 : n;
  }
  const long long cap_items = (long long)p.nb * p.n_heads *
                              (((long long)p.max_pages_per_seq * p.page_tokens + kMinItemTokens - 1) / kMinItemTokens);
  long long grid = (long long)resident * sm_count;
  if (grid > cap_items) grid = cap_items;
  if (grid < 1) grid = 1;
  attn_stored_mma_kernel<G, ROPE><<<(int)grid, kThreads, smem, stream>>>(k, v, k_run, v_run, p);
  return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& k_run, const CUtensorMap& v_run,
                     const StoredParams& p, int sm_count, cudaStream_t stream) {
  if (p.rope.cs != nullptr) return launch_g<G, true>(k, v, k_run, v_run, p, sm_count, stream);
  return launch_g<G, false>(k, v, k_run, v_run, p, sm_count, stream);
}

}  // namespace

bool stored_mma_supported(int dtype, int head_dim, int group, int max_batch) {
  if (dtype != ECHOKV_BF16 || head_dim != 128) return false;
  if (group != 1 && group != 2 && group != 4 && group != 8) return false;
  return max_batch <= kStoredMaxBatchPerLaunch * kStoredMaxLaunches;
}

int stored_rows_per_box(int page_tokens) { return page_tokens < kStageTokens ? page_tokens : kStageTokens; }

cudaError_t launch_attn_stored_mma(const AttnArgs& a, const CUtensorMap& k_map, const CUtensorMap& v_map,
                                   const CUtensorMap& k_run_map, const CUtensorMap& v_run_map, int n_heads, int32_t* item_tokens_slots, int sm_count, cudaStream_t stream) {
  if (n_heads == 0) return cudaSuccess;
  StoredParams p;
  p.q = reinterpret_cast<const __nv_bfloat16*>(a.q);
  p.slots = a.slots;
  p.lens = a.lens;
  p.table = a.geom.table;
  p.max_batch = a.geom.max_batch;
  p.max_pages_per_seq = a.geom.max_pages_per_seq;
  p.page_tokens = a.geom.page_tokens;
  p.n_pages = a.geom.n_pages;
  p.part_ml = a.parts.ml;
  p.part_o = a.parts.o;
  p.max_parts = a.parts.max_parts;
  p.status = a.status;
  p.n_q_heads = a.n_q_heads;
  p.n_heads = n_heads;
  p.rows_per_box = stored_rows_per_box(a.geom.page_tokens);
  p.scale_log2e = a.scale_log2e;
  p.rope = a.rope;
  const int g = a.n_q_heads / a.n_kv_heads;
  for (int b0 = 0, launch = 0; b0 < a.batch; b0 += kStoredMaxBatchPerLaunch, ++launch) {
    if (launch >= kStoredMaxLaunches) return cudaErrorInvalidValue;
    p.b0 = b0;
    p.nb = a.batch - b0 < kStoredMaxBatchPerLaunch ? a.batch - b0 : kStoredMaxBatchPerLaunch;
    p.item_tokens_out = item_tokens_slots + launch;
    cudaError_t e;
    switch (g) {
      case 1: e = launch_g<1>(k_map, v_map, k_run_map, v_run_map, p, sm_count, stream); break;
      case 2: e = launch_g<2>(k_map, v_map, k_run_map, v_run_map, p, sm_count, stream); break;
      case 4: e = launch_g<4>(k_map, v_map, k_run_map, v_run_map, p, sm_count, stream); break;
      case 8: e = launch_g<8>(k_map, v_map, k_run_map, v_run_map, p, sm_count, stream); break;
      default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace echokv
