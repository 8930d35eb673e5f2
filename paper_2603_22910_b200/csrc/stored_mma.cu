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
//
// With a rotation set (Section 3.2: the cache holds keys prior to the rotary embedding) the keys are turned to
// their positions as they are read.  That is ALU work of several hundred instructions per 16 tokens, too much
// for the four consumer warps beside their own work, so attn_stored_rope_kernel splits the roles: four score
// warps turn the keys (fp32, two frequency indices per instruction) and form q . k as tf32 products, hand the
// scores of a stage through shared memory to two value warps, which run the softmax and P V; two more warps
// issue the copies.
#include "stored_mma.h"

#include "ptx_sm100.cuh"

namespace echokv {

namespace {

constexpr int kStoredStages = 3;                     // stages of 32 KiB per CTA of the kernel without a rotation
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
constexpr int kThreads = 32 * (1 + kConsumers);          // a warp that issues the copies, four consumer warps
constexpr int kValueWarps = 2;                            // value warps of the rotating kernel: 64 output features each
constexpr int kRopeThreads = 32 * (kConsumers + kValueWarps + 2);  // rotating kernel: four score warps, the value
                                                         // warps, a warp that issues the K copies, one for the V copies
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
  int32_t* item_tokens_out;   // where this launch publishes its item_tokens (null: nobody asks)
  int b0, nb;                 // batch entries [b0, b0 + nb) are handled by this launch
  int n_q_heads, n_heads;     // query heads in all; stored KV heads attended (0 .. n_heads - 1)
  int rows_per_box;           // token rows per TMA box: min(page_tokens, 64)
  int page_shift, box_shift;  // log2 of page_tokens and of rows_per_box (both powers of two)
  float scale_log2e;
  RopeTable rope;             // read by the rotating kernels only
  // key_scores_rope_kernel only: where the scores go, and which tokens count as predicted
  float* scores;              // [batch][n_q_heads][l_cap]
  int l_cap, n_sink, n_window;
};

// What both kernels keep about the work items
struct StoredItems {
  int cum_items[kStoredMaxBatchPerLaunch + 1];
  unsigned long long total_tokens;
  int item_tokens;
  int abort_flag;
};

template <int G>
struct StoredSmemTail {
  float mo[kConsumers][G][128];
  float mm[kConsumers][8];
  float ml[kConsumers][8];
  StoredItems items;
  unsigned long long full_bar[kStoredStages];
  unsigned long long empty_bar[kStoredStages];
  uint32_t box_ok[kStoredStages];
};

// Barrier over the four consumer warps (128 threads, named barrier 1).
__device__ __forceinline__ void consumers_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// The same, also ANDing a flag (see the bounded waits).
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

__device__ __forceinline__ Item decode_item(const StoredItems& t, int item, int n_heads, int nb) {
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

// ---- set-up shared by both kernels: item size from the lengths present, items per sequence ---------------------
// Returns item_tokens; the number of items is t.cum_items[p.nb].  Called by every thread of the CTA, after thread 0
// has initialised the kernel's barriers (fenced here).
__device__ __forceinline__ int stored_setup(StoredItems& t, const StoredParams& p) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_threads = blockDim.x;
  const int capacity = p.max_pages_per_seq * p.page_tokens;
  if (tid == 0) {
    t.total_tokens = 0ull;
    t.abort_flag = 0;
    t.cum_items[0] = 0;
    mbar_fence_init();
  }
  __syncthreads();
  {
    unsigned long long mine = 0ull;
    for (int i = tid; i < p.nb; i += n_threads) {
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
    if (blockIdx.x == 0 && p.item_tokens_out != nullptr) *p.item_tokens_out = (int)per_item;
  }
  __syncthreads();
  const int item_tokens = t.item_tokens;
  for (int i = tid; i < p.nb; i += n_threads) {
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
  return item_tokens;
}

// ---- issuing the TMA copies ------------------------------------------------------------------------------------
// Lane l of the issuing warp owns box l of a stage (box row group l / 4; K lo, K hi, V lo, V hi = l % 4).
// A cursor stands on a stage of this CTA's stage sequence (the stages of its items, in the order the consumers take
// them) and holds this lane's block-table entry for it, requested when the cursor got there.
struct StageCursor {
  int item, j, n_iter, page, kvh, t_begin, t_end;
  const int32_t* table;
  bool more;            // the cursor stands on a stage (false: past the end)

  __device__ __forceinline__ void load_item(const StoredItems& t, const StoredParams& p, int item_tokens,
                                            int n_items) {
    if (item >= n_items) { more = false; return; }
    const Item w = decode_item(t, item, p.n_heads, p.nb);
    const int b = p.b0 + w.b;
    const int slot = p.slots ? p.slots[b] : b;
    kvh = w.kvh;
    t_begin = w.chunk * item_tokens;
    t_end = min(p.lens[b], t_begin + item_tokens);
    n_iter = (t_end - t_begin + kStageTokens - 1) / kStageTokens;      // >= 1: an item has a token
    table = p.table + (size_t)slot * p.max_pages_per_seq;
    j = 0;
  }
  // one stage forward
  __device__ __forceinline__ void advance(const StoredItems& t, const StoredParams& p, int item_tokens,
                                          int n_items) {
    if (!more) return;
    if (++j == n_iter) {
      item += gridDim.x;
      load_item(t, p, item_tokens, n_items);
    }
  }
  __device__ __forceinline__ void request_page(const StoredParams& p, int lane) {
    const int n_boxes = (kStageTokens >> p.box_shift) * 4;
    const int tb = t_begin + j * kStageTokens + ((lane >> 2) << p.box_shift);
    page = (more && lane < n_boxes && tb < t_end) ? table[tb >> p.page_shift] : -1;
  }
  // onto the first stage of the sequence
  __device__ __forceinline__ void init(const StoredItems& t, const StoredParams& p, int item_tokens, int n_items,
                                       int lane) {
    more = true;
    item = blockIdx.x;
    n_iter = j = kvh = t_begin = t_end = 0;
    table = p.table;
    load_item(t, p, item_tokens, n_items);
    request_page(p, lane);
  }
  // The stage the cursor stands on: row = pool row of this lane's box, -1 if the lane has none there, -2 if its page
  // id is out of range; head = the KV head.  Then one stage forward (its block-table entry is requested now and
  // used at the next call).  Call only while `more`.
  __device__ __forceinline__ void take(const StoredItems& t, const StoredParams& p, int item_tokens, int n_items,
                                       int lane, long long& row, int& head) {
    const int n_boxes = (kStageTokens >> p.box_shift) * 4;
    const int tb = t_begin + j * kStageTokens + ((lane >> 2) << p.box_shift);      // first token of this lane's box
    row = -1;
    if (lane < n_boxes && tb < t_end)
      row = (page < 0 || page >= p.n_pages) ? -2 : ((long long)page << p.page_shift) + (tb & (p.page_tokens - 1));
    head = kvh;
    advance(t, p, item_tokens, n_items);
    request_page(p, lane);
  }
};

// step() issues the copies of the next stage of the sequence; false once nothing is left or a wait gave up.
// KINDS: 3 = a stage holds K and V (32 KiB), 1 = the ring holds K halves only, 2 = V halves only (16 KiB each).
template <int NS, int KINDS>
struct StoredProducer {
  StageCursor cur;
  uint32_t n;           // the stage the cursor stands on = stages issued so far
  bool alive;

  __device__ __forceinline__ void init(const StoredItems& t, const StoredParams& p, int item_tokens, int n_items,
                                       int lane) {
    cur.init(t, p, item_tokens, n_items, lane);
    n = 0;
    alive = true;
  }
  // ring: shared address of slot 0; full / empty: the ring's barriers; box_ok: where the consumers find which boxes
  // of a slot hold cached tokens (nullptr: nobody asks)
  __device__ __forceinline__ bool step(const StoredItems& t, const StoredParams& p, const CUtensorMap* tm_k,
                                       const CUtensorMap* tm_v, const CUtensorMap* tm_k_run,
                                       const CUtensorMap* tm_v_run, uint32_t ring, unsigned long long* full_bar,
                                       unsigned long long* empty_bar, uint32_t* box_ok, volatile int* abort_flag,
                                       int item_tokens, int n_items, int lane) {
    if (!alive || !cur.more) return false;
    constexpr uint32_t kSlot = KINDS == 3 ? kStageBytes : kStageBytes / 2;
    constexpr uint32_t kLaneMask = KINDS == 3 ? 0xffffffffu : KINDS == 1 ? 0x33333333u : 0xccccccccu;
    const int rpb = p.rows_per_box, n_boxes = (kStageTokens >> p.box_shift) * 4;
    const int sub = lane >> 2, kind = lane & 3;
    const uint32_t s = n % NS;
    const uint32_t ph = (n / NS) & 1u;
    bool ok = true;
    if (lane == 0) ok = mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, abort_flag, p.status);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (!ok) { alive = false; return false; }
    long long row;
    int head;
    cur.take(t, p, item_tokens, n_items, lane, row, head);
    if (row == -2 && (KINDS & 1)) report(p.status, ECHOKV_EBADPAGE);
    const uint32_t ok_mask = __ballot_sync(0xffffffffu, row >= 0);
    // all boxes of the stage cached and consecutive in the pool: one 64-row copy per kind instead of one
    // per page (lanes 0..3 hold the first page's row for the four kinds)
    const long long row0 = __shfl_sync(0xffffffffu, row, kind);
    const bool run = n_boxes > 4 && __all_sync(0xffffffffu, lane >= n_boxes || (row >= 0 && row == row0 + sub * rpb));
    const uint32_t full = smem_u32(&full_bar[s]);
    if (lane == 0) {
      if (box_ok != nullptr) box_ok[s] = ok_mask;
      mbar_arrive_expect_tx(full, __popc(ok_mask & kLaneMask) * (uint32_t)rpb * 128u);
    }
    __syncwarp();
    // (lanes of kinds 0 and 2 copy: one box holds both feature halves, K or V)
    const bool mine = (kind == 0 && (KINDS & 1)) || (kind == 2 && (KINDS & 2));
    const uint32_t dst = ring + s * kSlot + (KINDS == 3 ? kind * kBlockBytes : 0);
    if (run) {
      if (lane < 4 && mine) tma_load_4d(dst, kind < 2 ? tm_k_run : tm_v_run, 0, 0, head * 2, (int)(row >> 3), full);
    } else if (row >= 0 && mine) {
      tma_load_4d(dst + sub * rpb * 256, kind < 2 ? tm_k : tm_v, 0, 0, head * 2, (int)(row >> 3), full);
    }
    ++n;
    return true;
  }
  // stopped with work left: a wait gave up
  __device__ __forceinline__ bool gave_up() const { return !alive && cur.more; }
  // let every copy this warp started land before the CTA leaves (earlier uses of a slot completed before a later
  // one could be issued, so the last stage per slot is enough)
  __device__ __forceinline__ void drain(unsigned long long* full_bar, int lane) const {
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < NS; ++k) {
        if (n > (uint32_t)k) {
          const uint32_t st = n - 1u - (uint32_t)k;
          mbar_drain(smem_u32(&full_bar[st % NS]), (st / NS) & 1u);
        }
      }
    }
  }
};

// ---- pieces of the consumer side ---------------------------------------------------------------------------------
// bit i: token i of the stage holds a cached token (ok_mask: which boxes were copied; n_tok: tokens of the item left)
__device__ __forceinline__ unsigned long long stage_mask(uint32_t ok_mask, int rpb, int n_tok) {
  const unsigned long long in_len = n_tok >= 64 ? ~0ull : ((1ull << n_tok) - 1ull);
  unsigned long long in_box = 0ull;
  const unsigned long long box_bits = rpb >= 64 ? ~0ull : ((1ull << rpb) - 1ull);
  for (int g = 0; g < kStageTokens / rpb; ++g)
    if ((ok_mask >> (g * 4)) & 1u) in_box |= box_bits << (g * rpb);
  return in_len & in_box;
}

// A (or B) fragments of Q for query head lane / 4 of KV head kvh: packed feature pairs 16 ks + qd (+1) and
// 16 ks + 8 + qd (+1), qd = 2 (lane % 4); zero for rows past the group.
template <int G>
__device__ __forceinline__ void load_q_fragments(const StoredParams& p, int b, int kvh, int lane, uint32_t (&qa0)[8],
                                                 uint32_t (&qa2)[8]) {
  const int row = lane >> 2, qd = (lane & 3) * 2;
  const __nv_bfloat16* qrow = p.q + ((size_t)b * p.n_q_heads + (size_t)kvh * G + row) * 128 + qd;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    qa0[ks] = row < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16) : 0u;
    qa2[ks] = row < G ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8) : 0u;
  }
}

// =================================================================================================================
// Keys used as stored (no rotation)
// =================================================================================================================
template <int G>
__global__ void __launch_bounds__(kThreads, 2)
attn_stored_mma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       const __grid_constant__ CUtensorMap tm_k_run, const __grid_constant__ CUtensorMap tm_v_run,
                       const StoredParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  constexpr int NS = kStoredStages;
  StoredSmemTail<G>& t = *reinterpret_cast<StoredSmemTail<G>*>(smem + NS * kStageBytes);
  const uint32_t stage_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &t.items.abort_flag;
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(smem_u32(&t.full_bar[s]), 1);
      mbar_init(smem_u32(&t.empty_bar[s]), kConsumers);
    }
  }
  const int item_tokens = stored_setup(t.items, p);
  const int n_items = t.items.cum_items[p.nb];
  const int rpb = p.rows_per_box;

  if (warp == 0) {
    // =============================== TMA producer ===============================================
    StoredProducer<NS, 3> pr;
    pr.init(t.items, p, item_tokens, n_items, lane);
    while (pr.step(t.items, p, &tm_k, &tm_v, &tm_k_run, &tm_v_run, stage_base, t.full_bar, t.empty_bar, t.box_ok,
                   abort_flag, item_tokens, n_items, lane)) {
    }
    if (pr.gave_up()) pr.drain(t.full_bar, lane);
  } else {
    // =============================== consumers (4 warps) ========================================
    const int cw = warp - 1;
    const int row = lane >> 2;                // query head of the group held in c0 / c1
    const int qd = (lane & 3) * 2;            // first of this thread's two columns inside an 8-wide tile
    const int ct = tid - 32;                  // 0..127: output feature at the item-end merge
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Item w = decode_item(t.items, item, p.n_heads, p.nb);
      const int b = p.b0 + w.b;
      const int len = p.lens[b];
      const int t_begin = w.chunk * item_tokens;
      const int t_end = min(len, t_begin + item_tokens);
      const int n_iter = (t_end - t_begin + kStageTokens - 1) / kStageTokens;

      // A fragments of Q: rows 0..G-1 are the group's query heads, the rest is zero
      uint32_t qa0[8], qa2[8];
      load_q_fragments<G>(p, b, w.kvh, lane, qa0, qa2);
      float m_run = -INFINITY, l_run = 0.f;
      float o[16][4];
#pragma unroll
      for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;

      for (int j = 0; j < n_iter; ++j, ++it) {
        const uint32_t s = it % NS;
        const uint32_t ph = (it / NS) & 1u;
        const bool got = mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
        const uint32_t sb = stage_base + s * kStageBytes;
        const int t0 = t_begin + j * kStageTokens;
        // bit i: token i of this warp's 16-token slice of the stage holds a cached token
        const uint32_t vmask =
            (uint32_t)(stage_mask(t.box_ok[s], rpb, min(kStageTokens, t_end - t0)) >> (cw * kWarpTokens)) & 0xffffu;
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
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const int c0 = (ks & 3) * 2 + ((lane >> 3) & 1);
            uint32_t r0, r1, r2, r3;
            ldsm_x4(sb + stage_off(tok_k, (ks >> 2) * 8 + c0), r0, r1, r2, r3);
            mma_m16n8k16_bf16(sc[0], qa0[ks], 0u, qa2[ks], 0u, r0, r1);
            mma_m16n8k16_bf16(sc[1], qa0[ks], 0u, qa2[ks], 0u, r2, r3);
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

// =================================================================================================================
// Keys rotated to their positions as they are read (Section 3.2)
// =================================================================================================================
// The angle of token 16 u + r is the sum of a coarse angle (row u of the coarse table) and a fine one (row r of the
// fine table), and q . R(u, r) k = (R(u)^T q) . (R(r) k): the queries are turned back by the coarse angle of the
// 16-token slice, a key is turned by one of 16 fine angles.  Frequency index f pairs feature f of the head's first
// 64 features with feature f + 64.
//
// Roles.  Score warp w (warps 0..3) takes tokens 16 w .. 16 w + 15 of every stage: keys turned in fp32, q . k as
// tf32 products, the 16 x G raw scores into a buffer in shared memory.  Value warp w (warps 4, 5) takes features
// 64 w .. 64 w + 63 of the output for all 64 tokens of the stage: both value warps run the same softmax over the
// stage's scores (same operations, same results) and multiply P into their slice of V, so the running output needs
// 32 registers and nothing is combined across warps at the end of an item.  Warp 6 issues the K copies, warp 7 the
// V copies: the per-stage block-table arithmetic is a serial chain of some hundred instructions that must not sit
// in a warp the others wait for.
//
// K and V travel in rings of their own (16 KiB slots: 64 tokens x 128 features): a K slot comes free as soon as the
// score warps have turned its keys, a V slot when the value warps are done with it.
constexpr int kFineRowPairs = 72;     // index pairs per row of the in-CTA fine table: 64 + 8 of padding, so that the
                                      // 16-byte reads of two successive rows fill the 32 banks exactly
constexpr int kScoreStride = 72;      // floats per query head in a score buffer: 64 tokens + 8 of padding
// Six slots fit beside the tables with two CTAs on an SM (five when the score buffers hold eight heads).
constexpr int kRopeKSlots = 3;
template <int G> struct RopeVSlots { static constexpr int value = G >= 8 ? 2 : 3; };
constexpr int kRingMax = 4;
constexpr int kSlotBytes = 2 * kBlockBytes;

// The score warps' work on one 16-token slice of a K slot (sb: the slot; tok_k: this lane's ldmatrix row):
// S^T = K' Q'^T as tf32 products m16n8k8 with the 16 tokens on the M rows (K': keys turned by the fine angle; Q':
// queries turned back by the slice's coarse angle, coarse_q): the thread's two features of a token (f and f + 1) are
// the k indices lane % 4 and lane % 4 + 4 of one product, for the key and for the query alike.  The features
// 64 .. 127 accumulate apart: two shorter chains of products.
// acc[0], acc[1]: token lane / 4 of the slice, heads qd and qd + 1; acc[2], acc[3]: token lane / 4 + 8 (raw q . k).
__device__ __forceinline__ void rotated_key_scores(uint32_t sb, int tok_k, const float4* coarse_q,
                                                   const float4* fine_a, const float4* fine_b,
                                                   const uint32_t (&qa0)[8], const uint32_t (&qa2)[8], int lane,
                                                   float (&acc)[4]) {
  float acc_lo[4] = {0.f, 0.f, 0.f, 0.f}, acc_hi[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int ks = 0; ks < 4; ++ks) {
    // register i: token tile i >> 1 (slice offsets lane / 4 and lane / 4 + 8), frequency indices
    // f = 16 ks + 8 (i & 1) + qd and f + 1; ka the features f, kb the features f + 64
    const int c0 = ks * 2 + ((lane >> 3) & 1);
    uint32_t ka[4], kb[4];
    ldsm_x4(sb + stage_off(tok_k, c0), ka[0], ka[1], ka[2], ka[3]);
    ldsm_x4(sb + stage_off(tok_k, 8 + c0), kb[0], kb[1], kb[2], kb[3]);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      // the queries' features f, f + 1 (qa) and f + 64, f + 65 (qb), turned BACK by the slice's coarse angle:
      // q . R(U + r) k = (R(U)^T q) . (R(r) k), so a key is turned by one of the 16 fine angles only
      const float4 bw = coarse_q[ks * 8 + h * 4];                         // (cos f, sin f, cos f+1, sin f+1)
      const float2 bc = make_float2(bw.x, bw.z), bs = make_float2(bw.y, bw.w);
      const uint32_t q_lo = h ? qa2[ks] : qa0[ks];
      const uint32_t q_hi = h ? qa2[ks + 4] : qa0[ks + 4];
      const float2 qa = make_float2(bf16_lo(q_lo), bf16_hi(q_lo)), qb = make_float2(bf16_lo(q_hi), bf16_hi(q_hi));
      const float2 ta = __ffma2_rn(bs, qb, __fmul2_rn(bc, qa));
      float2 tb = __fmul2_rn(bc, qb);
      tb.x = fmaf(-bs.x, qa.x, tb.x);
      tb.y = fmaf(-bs.y, qa.y, tb.y);
      float2 lo[2], hi[2];
#pragma unroll
      for (int tile = 0; tile < 2; ++tile) {
        const int i = tile * 2 + h;
        const float4 fw = (tile ? fine_b : fine_a)[ks * 8 + h * 4];       // (cos f, cos f+1, sin f, sin f+1)
        const float2 fc = make_float2(fw.x, fw.y), fs = make_float2(fw.z, fw.w);
        const float2 xa = make_float2(bf16_lo(ka[i]), bf16_hi(ka[i]));
        const float2 xb = make_float2(bf16_lo(kb[i]), bf16_hi(kb[i]));
        lo[tile] = __fmul2_rn(xa, fc);
        lo[tile].x = fmaf(-xb.x, fs.x, lo[tile].x);
        lo[tile].y = fmaf(-xb.y, fs.y, lo[tile].y);
        hi[tile] = __ffma2_rn(xa, fs, __fmul2_rn(xb, fc));
      }
      // (the tensor core chops its operands to tf32: the turned queries are rounded to nearest first, eight values
      // per step against the 32 of the keys, which halves the error the chopping leaves in the scores)
      mma_m16n8k8_tf32(acc_lo, __float_as_uint(lo[0].x), __float_as_uint(lo[1].x), __float_as_uint(lo[0].y),
                       __float_as_uint(lo[1].y), to_tf32(ta.x), to_tf32(ta.y));
      mma_m16n8k8_tf32(acc_hi, __float_as_uint(hi[0].x), __float_as_uint(hi[1].x), __float_as_uint(hi[0].y),
                       __float_as_uint(hi[1].y), to_tf32(tb.x), to_tf32(tb.y));
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) acc[e] = acc_lo[e] + acc_hi[e];
}

// The fine table into shared memory: entry (r, f even) = (cos f, cos f+1, sin f, sin f+1) of offset r.
__device__ __forceinline__ void load_fine_table(float2* fine, const RopeTable& rope) {
  for (int i = threadIdx.x; i < kRopeFineRows * 64; i += blockDim.x) {
    const float2 cs = rope.fine[i];
    float* entry = reinterpret_cast<float*>(fine + (i >> 6) * kFineRowPairs + (i & 62));
    entry[i & 1] = cs.x;
    entry[2 + (i & 1)] = cs.y;
  }
}

template <int G>
struct StoredRopeSmem {
  // entry (r, f even): (cos f, cos f+1, sin f, sin f+1) of offset r; one entry = two float2
  float2 fine[kRopeFineRows * kFineRowPairs];
  float2 coarse[kConsumers][64];                  // per score warp: the coarse row of the slice it works on
  float scores[2][G * kScoreStride];              // two deep: raw q . k of the stage's 64 tokens x G heads
  StoredItems items;
  unsigned long long s_full[2];                   // score warps -> value warps: the buffer holds a stage's scores
  unsigned long long s_empty[2];                  // value warps -> score warps: the buffer has been read
  unsigned long long k_full[kRingMax], k_empty[kRingMax];
  unsigned long long v_full[kRingMax], v_empty[kRingMax];
  uint32_t box_ok[kRingMax];                      // per V slot: which boxes hold cached tokens
};

template <int G>
__global__ void __launch_bounds__(kRopeThreads, 2)
attn_stored_rope_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                        const __grid_constant__ CUtensorMap tm_k_run, const __grid_constant__ CUtensorMap tm_v_run,
                        const StoredParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  constexpr int NK = kRopeKSlots, NV = RopeVSlots<G>::value;
  StoredRopeSmem<G>& rs = *reinterpret_cast<StoredRopeSmem<G>*>(smem + (NK + NV) * kSlotBytes);
  const uint32_t k_ring = smem_u32(smem), v_ring = k_ring + NK * kSlotBytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &rs.items.abort_flag;
  load_fine_table(rs.fine, p.rope);
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&rs.s_full[i]), kConsumers);
      mbar_init(smem_u32(&rs.s_empty[i]), kValueWarps);
    }
    for (int i = 0; i < kRingMax; ++i) {
      mbar_init(smem_u32(&rs.k_full[i]), 1);
      mbar_init(smem_u32(&rs.k_empty[i]), kConsumers);
      mbar_init(smem_u32(&rs.v_full[i]), 1);
      mbar_init(smem_u32(&rs.v_empty[i]), kValueWarps);
    }
  }
  const int item_tokens = stored_setup(rs.items, p);
  const int n_items = rs.items.cum_items[p.nb];
  const int rpb = p.rows_per_box;
  const int cw = warp < kConsumers ? warp : warp - kConsumers;      // score warp: its token slice; value warp: its feature slice
  const int row = lane >> 2;                // MMA row / column of this thread: a token (scores) or a query head
  const int qd = (lane & 3) * 2;

  if (warp < kConsumers) {
    // =============================== score warps =================================================
    float2* coarse_w = rs.coarse[cw];
    const float4* coarse_q = reinterpret_cast<const float4*>(coarse_w + qd);
    const float4* fine_a = reinterpret_cast<const float4*>(rs.fine + row * kFineRowPairs + qd);
    const float4* fine_b = reinterpret_cast<const float4*>(rs.fine + (row + 8) * kFineRowPairs + qd);
    const int tok_k = cw * kWarpTokens + (lane >> 4) * 8 + (lane & 7);          // K rows: ldmatrix
    // one coarse row (64 index pairs, 512 bytes) into this warp's buffer, 16 bytes per lane
    auto fetch_coarse = [&](int stage_t0) {
      const int u = min(stage_t0 / kRopeFineRows + cw, p.rope.stride / kRopeFineRows - 1);
      __syncwarp();          // every lane has read the row that is there now
      asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_u32(coarse_w + lane * 2)),
                   "l"(p.rope.coarse + (size_t)u * 64 + lane * 2)
                   : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Item w = decode_item(rs.items, item, p.n_heads, p.nb);
      const int b = p.b0 + w.b;
      const int t_begin = w.chunk * item_tokens;
      const int t_end = min(p.lens[b], t_begin + item_tokens);
      const int n_iter = (t_end - t_begin + kStageTokens - 1) / kStageTokens;
      // B fragments of Q: column lane / 4 is a query head of the group (zero past the group)
      uint32_t qa0[8], qa2[8];
      load_q_fragments<G>(p, b, w.kvh, lane, qa0, qa2);
      fetch_coarse(t_begin);
      for (int j = 0; j < n_iter; ++j, ++it) {
        const uint32_t s = it % NK;
        const uint32_t slot = it & 1u;
        bool got = mbar_wait(smem_u32(&rs.k_full[s]), (it / NK) & 1u, abort_flag, p.status);
        got = got && mbar_wait(smem_u32(&rs.s_empty[slot]), ((it >> 1) & 1u) ^ 1u, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
        const uint32_t sb = k_ring + s * kSlotBytes;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();            // this slice's coarse row is in the warp's buffer
        float acc[4];
        rotated_key_scores(sb, tok_k, coarse_q, fine_a, fine_b, qa0, qa2, lane, acc);
        // acc[0], acc[1]: token lane / 4 of the slice, heads qd and qd + 1; acc[2], acc[3]: token lane / 4 + 8
        float* sbuf = rs.scores[slot] + cw * kWarpTokens + row;
        if (qd < G) {
          sbuf[qd * kScoreStride] = acc[0];
          sbuf[qd * kScoreStride + 8] = acc[2];
        }
        if (qd + 1 < G) {
          sbuf[(qd + 1) * kScoreStride] = acc[1];
          sbuf[(qd + 1) * kScoreStride + 8] = acc[3];
        }
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(smem_u32(&rs.s_full[slot]));
          mbar_arrive(smem_u32(&rs.k_empty[s]));
        }
        if (j + 1 < n_iter) fetch_coarse(t_begin + (j + 1) * kStageTokens);   // in flight until the next slice
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");   // (a copy started before a wait gave up)
  } else if (warp == kConsumers + kValueWarps) {
    // =============================== the warp that issues the K copies ===========================
    StoredProducer<NK, 1> pr;
    pr.init(rs.items, p, item_tokens, n_items, lane);
    while (pr.step(rs.items, p, &tm_k, &tm_v, &tm_k_run, &tm_v_run, k_ring, rs.k_full, rs.k_empty, nullptr, abort_flag,
                   item_tokens, n_items, lane)) {
    }
    if (pr.gave_up()) pr.drain(rs.k_full, lane);
  } else if (warp == kConsumers + kValueWarps + 1) {
    // =============================== the warp that issues the V copies ===========================
    StoredProducer<NV, 2> pr;
    pr.init(rs.items, p, item_tokens, n_items, lane);
    while (pr.step(rs.items, p, &tm_k, &tm_v, &tm_k_run, &tm_v_run, v_ring, rs.v_full, rs.v_empty, rs.box_ok,
                   abort_flag, item_tokens, n_items, lane)) {
    }
    if (pr.gave_up()) pr.drain(rs.v_full, lane);
  } else {
    // =============================== value warps =================================================
    constexpr int kPieces = 16 / kValueWarps;   // 16-byte pieces (8 features) of this warp's slice of V
    constexpr int kTiles = kPieces;             // 8-feature output tiles of the slice
    const int f0 = cw * kPieces;
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Item w = decode_item(rs.items, item, p.n_heads, p.nb);
      const int b = p.b0 + w.b;
      const int t_begin = w.chunk * item_tokens;
      const int t_end = min(p.lens[b], t_begin + item_tokens);
      const int n_iter = (t_end - t_begin + kStageTokens - 1) / kStageTokens;
      float m_run = -INFINITY, l_run = 0.f;
      float o[kTiles][4];
#pragma unroll
      for (int nt = 0; nt < kTiles; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;

      for (int j = 0; j < n_iter; ++j, ++it) {
        const uint32_t s = it % NV;
        const uint32_t slot = it & 1u;
        bool got = mbar_wait(smem_u32(&rs.v_full[s]), (it / NV) & 1u, abort_flag, p.status);
        got = got && mbar_wait(smem_u32(&rs.s_full[slot]), (it >> 1) & 1u, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
        const uint32_t vb = v_ring + s * kSlotBytes;
        const int t0 = t_begin + j * kStageTokens;
        // scores of query head `row`: sc[kk][2 h + e] = token 16 kk + 8 h + qd + e of the stage
        float sc[4][4];           // (rows past the group: zeros, their results are never written)
        {
          const float* sbuf = rs.scores[slot] + (row < G ? row : 0) * kScoreStride + qd;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const float2 s0 = *reinterpret_cast<const float2*>(sbuf + kk * 16);
            const float2 s1 = *reinterpret_cast<const float2*>(sbuf + kk * 16 + 8);
            sc[kk][0] = row < G ? s0.x : 0.f;
            sc[kk][1] = row < G ? s0.y : 0.f;
            sc[kk][2] = row < G ? s1.x : 0.f;
            sc[kk][3] = row < G ? s1.y : 0.f;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&rs.s_empty[slot]));
        const unsigned long long valid = stage_mask(rs.box_ok[s], rpb, min(kStageTokens, t_end - t0));
        if (valid != 0ull) {
          const bool all_valid = valid == ~0ull;
          if (!all_valid) {
            // rows without a cached token may hold anything (never written, or a skipped page): zero this warp's
            // slice of them in V so that 0 * V stays 0; their scores are masked below
            for (int idx = lane; idx < kStageTokens * kPieces; idx += 32) {
              const int r = idx / kPieces;
              if (!((valid >> r) & 1ull)) {
                const uint32_t a = vb + stage_off(r, f0 + idx % kPieces);
                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0u) : "memory");
              }
            }
            __syncwarp();
          }
          // ---- online softmax on row `row` over the stage's 64 tokens (the same in all four warps) ----
          float mx = -INFINITY;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float v = sc[kk][e] * p.scale_log2e;
              if (!all_valid && !((valid >> (kk * 16 + (e >> 1) * 8 + qd + (e & 1))) & 1ull)) v = -INFINITY;
              sc[kk][e] = v;
              mx = fmaxf(mx, v);
            }
          }
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
          const float m_new = fmaxf(m_run, mx);     // finite: the stage has a valid token
          const float alpha = exp2f(m_run - m_new);
          m_run = m_new;
          uint32_t p_hi[4][2], p_lo[4][2];          // [kk][h]: P = P_hi + P_lo, each a packed bf16 pair
          float psum = 0.f;
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const float p0 = exp2f(sc[kk][2 * h] - m_new);
              const float p1 = exp2f(sc[kk][2 * h + 1] - m_new);
              psum += p0 + p1;
              const __nv_bfloat162 hh = __floats2bfloat162_rn(p0, p1);
              p_hi[kk][h] = *reinterpret_cast<const uint32_t*>(&hh);
              p_lo[kk][h] = pack_bf16(p0 - __low2float(hh), p1 - __high2float(hh));
            }
          }
          l_run = l_run * alpha + psum;
          if (alpha != 1.f) {     // (the quad shares alpha)
#pragma unroll
            for (int nt = 0; nt < kTiles; ++nt)
#pragma unroll
              for (int e = 0; e < 4; ++e) o[nt][e] *= alpha;
          }
          // ---- O += P V on this warp's 32 features: rows 0..7 take P_hi, rows 8..15 take P_lo ----
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const int tok_v = kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);    // V rows: ldmatrix.trans
#pragma unroll
            for (int dp = 0; dp < kTiles / 2; ++dp) {
              uint32_t r0, r1, r2, r3;
              ldsm_x4_trans(vb + stage_off(tok_v, f0 + 2 * dp + (lane >> 4)), r0, r1, r2, r3);
              mma_m16n8k16_bf16(o[2 * dp], p_hi[kk][0], p_lo[kk][0], p_hi[kk][1], p_lo[kk][1], r0, r1);
              mma_m16n8k16_bf16(o[2 * dp + 1], p_hi[kk][0], p_lo[kk][0], p_hi[kk][1], p_lo[kk][1], r2, r3);
            }
          }
          if (!all_valid) fence_proxy_async_smem();   // the zeroed rows, before TMA writes there again
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&rs.v_empty[s]));
      }
      if (!alive) break;

      // ---- item end: this warp's 32 features of the partial, straight from the registers ----
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
      l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
      if (row < G) {
        const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)w.kvh * G + row) * p.max_parts + w.chunk;
#pragma unroll
        for (int nt = 0; nt < kTiles; ++nt)
          *reinterpret_cast<float2*>(p.part_o + pidx * 128 + cw * (8 * kTiles) + nt * 8 + qd) =
              make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
        if (cw == 0 && (lane & 3) == 0) p.part_ml[pidx] = make_float2(m_run, l_run);
      }
    }
  }
}

// =================================================================================================================
// Scores only: S[b][h][t] = q_h . R_t k_t (base-2 units) for the query heads of stored KV heads, written to memory
// =================================================================================================================
// What the absorbed V side needs when the K side has to be explicit (rotated keys): the score warps of the kernel
// above on a K ring alone -- four score warps and a warp that issues the copies.  Token slots of a sequence's whole
// 256-token tiles that hold no predicted token (sink / window tokens, tokens past the length, a page that could not
// be read) get -inf.
constexpr int kScoresThreads = 32 * (kConsumers + 1);
constexpr int kScoresKSlots = 3;            // three CTAs per SM: the score warps are what this kernel is short of

struct KeyScoresSmem {
  float2 fine[kRopeFineRows * kFineRowPairs];
  float2 coarse[kConsumers][64];
  StoredItems items;
  unsigned long long k_full[kScoresKSlots], k_empty[kScoresKSlots];
  uint32_t box_ok[kScoresKSlots];
};

template <int G>
__global__ void __launch_bounds__(kScoresThreads, 3)
key_scores_rope_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_k_run,
                       const StoredParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  constexpr int NK = kScoresKSlots;
  KeyScoresSmem& rs = *reinterpret_cast<KeyScoresSmem*>(smem + NK * kSlotBytes);
  const uint32_t k_ring = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &rs.items.abort_flag;
  load_fine_table(rs.fine, p.rope);
  if (tid == 0) {
    for (int i = 0; i < NK; ++i) {
      mbar_init(smem_u32(&rs.k_full[i]), 1);
      mbar_init(smem_u32(&rs.k_empty[i]), kConsumers);
    }
  }
  const int item_tokens = stored_setup(rs.items, p);
  const int n_items = rs.items.cum_items[p.nb];
  const int rpb = p.rows_per_box;

  if (warp == kConsumers) {
    // =============================== the warp that issues the K copies ===========================
    StoredProducer<NK, 1> pr;
    pr.init(rs.items, p, item_tokens, n_items, lane);
    while (pr.step(rs.items, p, &tm_k, &tm_k, &tm_k_run, &tm_k_run, k_ring, rs.k_full, rs.k_empty, rs.box_ok, abort_flag,
                   item_tokens, n_items, lane)) {
    }
    if (pr.gave_up()) pr.drain(rs.k_full, lane);
  } else {
    // =============================== score warps =================================================
    const int cw = warp;
    const int row = lane >> 2, qd = (lane & 3) * 2;
    float2* coarse_w = rs.coarse[cw];
    const float4* coarse_q = reinterpret_cast<const float4*>(coarse_w + qd);
    const float4* fine_a = reinterpret_cast<const float4*>(rs.fine + row * kFineRowPairs + qd);
    const float4* fine_b = reinterpret_cast<const float4*>(rs.fine + (row + 8) * kFineRowPairs + qd);
    const int tok_k = cw * kWarpTokens + (lane >> 4) * 8 + (lane & 7);          // K rows: ldmatrix
    auto fetch_coarse = [&](int stage_t0) {
      const int u = min(stage_t0 / kRopeFineRows + cw, p.rope.stride / kRopeFineRows - 1);
      __syncwarp();          // every lane has read the row that is there now
      asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_u32(coarse_w + lane * 2)),
                   "l"(p.rope.coarse + (size_t)u * 64 + lane * 2)
                   : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    uint32_t it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const Item w = decode_item(rs.items, item, p.n_heads, p.nb);
      const int b = p.b0 + w.b;
      const int len = p.lens[b];
      const int t_begin = w.chunk * item_tokens;
      const int t_end = min(len, t_begin + item_tokens);
      const int n_iter = (t_end - t_begin + kStageTokens - 1) / kStageTokens;
      const int pred_lo = predicted_lo(len, p.n_sink), pred_hi = predicted_hi(len, p.n_sink, p.n_window);
      const int write_end = min((len + 255) / 256 * 256, p.l_cap);     // whole 256-token tiles are written, no more
      float* s_rows = p.scores + ((size_t)b * p.n_q_heads + (size_t)w.kvh * G) * p.l_cap;
      uint32_t qa0[8], qa2[8];
      load_q_fragments<G>(p, b, w.kvh, lane, qa0, qa2);
      fetch_coarse(t_begin);
      for (int j = 0; j < n_iter; ++j, ++it) {
        const uint32_t s = it % NK;
        const bool got = mbar_wait(smem_u32(&rs.k_full[s]), (it / NK) & 1u, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, got)) { alive = false; break; }
        const uint32_t sb = k_ring + s * kSlotBytes;
        const int t0 = t_begin + j * kStageTokens;
        const unsigned long long valid = stage_mask(rs.box_ok[s], rpb, min(kStageTokens, t_end - t0));
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();            // this slice's coarse row is in the warp's buffer
        float acc[4];
        rotated_key_scores(sb, tok_k, coarse_q, fine_a, fine_b, qa0, qa2, lane, acc);
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&rs.k_empty[s]));
        if (j + 1 < n_iter) fetch_coarse(t0 + kStageTokens);
        // acc[0], acc[1]: token `row` of the slice, heads qd and qd + 1; acc[2], acc[3]: token row + 8
#pragma unroll
        for (int h8 = 0; h8 < 2; ++h8) {
          const int ts = cw * kWarpTokens + h8 * 8 + row, t = t0 + ts;
          const bool keep = ((valid >> ts) & 1ull) && t >= pred_lo && t < pred_hi;
          if (t < write_end) {
            if (qd < G) s_rows[(size_t)qd * p.l_cap + t] = keep ? acc[2 * h8] * p.scale_log2e : -INFINITY;
            if (qd + 1 < G) s_rows[(size_t)(qd + 1) * p.l_cap + t] = keep ? acc[2 * h8 + 1] * p.scale_log2e : -INFINITY;
          }
        }
        if (t0 + kStageTokens >= len) {
          // the sequence's last stage: the rest of its last 256-token tile holds no token
          for (int t = t0 + kStageTokens + cw * 32 + lane; t < write_end; t += kConsumers * 32)
#pragma unroll
            for (int gi = 0; gi < G; ++gi) s_rows[(size_t)gi * p.l_cap + t] = -INFINITY;
        }
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");   // (a copy started before a wait gave up)
  }
}

template <int G>
cudaError_t launch_scores_g(const CUtensorMap& k, const CUtensorMap& k_run, const StoredParams& p, int sm_count,
                            cudaStream_t stream) {
  const size_t smem = 1024 + (size_t)kScoresKSlots * kSlotBytes + sizeof(KeyScoresSmem);
  cudaError_t e = cudaFuncSetAttribute(key_scores_rope_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  static int resident = 0;   // per instantiation; the answer depends only on the kernel and the device type
  if (resident == 0) {
    int n = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, key_scores_rope_kernel<G>, kScoresThreads, smem);
    if (e != cudaSuccess) return e;
    resident = n < 1 ? 1 : n;
  }
  const long long cap_items = (long long)p.nb * p.n_heads *
                              (((long long)p.max_pages_per_seq * p.page_tokens + kMinItemTokens - 1) / kMinItemTokens);
  long long grid = (long long)resident * sm_count;
  if (grid > cap_items) grid = cap_items;
  if (grid < 1) grid = 1;
  key_scores_rope_kernel<G><<<(int)grid, kScoresThreads, smem, stream>>>(k, k_run, p);
  return cudaGetLastError();
}

template <int G, bool ROPE>
constexpr size_t stored_smem_bytes() {
  return 1024 + (ROPE ? (size_t)(kRopeKSlots + RopeVSlots<G>::value) * kSlotBytes + sizeof(StoredRopeSmem<G>)
                      : (size_t)kStoredStages * kStageBytes + sizeof(StoredSmemTail<G>));
}

template <int G, bool ROPE>
cudaError_t launch_g(const CUtensorMap& k, const CUtensorMap& v, const CUtensorMap& k_run, const CUtensorMap& v_run,
                     const StoredParams& p, int sm_count, cudaStream_t stream) {
  const size_t smem = stored_smem_bytes<G, ROPE>();
  const auto kernel = ROPE ? attn_stored_rope_kernel<G> : attn_stored_mma_kernel<G>;
  const int threads = ROPE ? kRopeThreads : kThreads;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // as many CTAs as stay resident, but never more than the items there can be
  static int resident = 0;   // per instantiation; the answer depends only on the kernel and the device type
  if (resident == 0) {
    int n = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, smem);
    if (e != cudaSuccess) return e;
    resident = n < 1 ? 1 : n;
  }
  const long long cap_items = (long long)p.nb * p.n_heads *
                              (((long long)p.max_pages_per_seq * p.page_tokens + kMinItemTokens - 1) / kMinItemTokens);
  long long grid = (long long)resident * sm_count;
  if (grid > cap_items) grid = cap_items;
  if (grid < 1) grid = 1;
  kernel<<<(int)grid, threads, smem, stream>>>(k, v, k_run, v_run, p);
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

namespace {
StoredParams stored_params(const AttnArgs& a, int n_heads) {
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
  p.item_tokens_out = nullptr;
  p.b0 = 0;
  p.nb = 0;
  p.n_q_heads = a.n_q_heads;
  p.n_heads = n_heads;
  p.rows_per_box = stored_rows_per_box(a.geom.page_tokens);
  p.page_shift = 0;
  while ((1 << p.page_shift) < p.page_tokens) ++p.page_shift;
  p.box_shift = 0;
  while ((1 << p.box_shift) < p.rows_per_box) ++p.box_shift;
  p.scale_log2e = a.scale_log2e;
  p.rope = a.rope;
  p.scores = nullptr;
  p.l_cap = p.n_sink = p.n_window = 0;
  return p;
}
}  // namespace

cudaError_t launch_attn_stored_mma(const AttnArgs& a, const CUtensorMap& k_map, const CUtensorMap& v_map,
                                   const CUtensorMap& k_run_map, const CUtensorMap& v_run_map, int n_heads, int32_t* item_tokens_slots, int sm_count, cudaStream_t stream) {
  if (n_heads == 0) return cudaSuccess;
  StoredParams p = stored_params(a, n_heads);
  if ((1 << p.page_shift) != p.page_tokens) return cudaErrorInvalidValue;     // (pages of 16, 32, 64 or 128 tokens)
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

cudaError_t launch_key_scores_stored(const AttnArgs& a, const CUtensorMap& k_map, const CUtensorMap& k_run_map,
                                     int n_heads, float* S, int l_cap, int n_sink, int n_window, int sm_count,
                                     cudaStream_t stream) {
  if (n_heads == 0) return cudaSuccess;
  if (a.dtype != ECHOKV_BF16 || a.head_dim != 128 || a.rope.cs == nullptr) return cudaErrorInvalidValue;
  StoredParams p = stored_params(a, n_heads);
  if ((1 << p.page_shift) != p.page_tokens) return cudaErrorInvalidValue;
  p.scores = S;
  p.l_cap = l_cap;
  p.n_sink = n_sink;
  p.n_window = n_window;
  const int g = a.n_q_heads / a.n_kv_heads;
  for (int b0 = 0; b0 < a.batch; b0 += kStoredMaxBatchPerLaunch) {
    p.b0 = b0;
    p.nb = a.batch - b0 < kStoredMaxBatchPerLaunch ? a.batch - b0 : kStoredMaxBatchPerLaunch;
    cudaError_t e;
    switch (g) {
      case 1: e = launch_scores_g<1>(k_map, k_run_map, p, sm_count, stream); break;
      case 2: e = launch_scores_g<2>(k_map, k_run_map, p, sm_count, stream); break;
      case 4: e = launch_scores_g<4>(k_map, k_run_map, p, sm_count, stream); break;
      case 8: e = launch_scores_g<8>(k_map, k_run_map, p, sm_count, stream); break;
      default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace echokv
