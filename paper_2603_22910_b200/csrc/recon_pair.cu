// Fused reconstruct-then-attend on CTA pairs (tcgen05 cta_group::2, sm_100a).
//
// The same computation as recon_tc.cu (Eq. 3 on the tensor cores, Eq. 7 on the accumulators), laid
// out over two SMs that run as one M = 256 tensor-core unit:
//
//   work item  = (sequence b, tile of 256 tokens, pair of dropped heads), one per CTA pair;
//                CTA r of the pair owns tokens [128 r, 128 r + 128) of the tile and head r of the pair
//   stage      = per CTA 128 token rows and the 128 predictor rows of its head, two 64-feature chunks
//                of each (64 KiB, 3 deep); every MMA reads the token rows of both CTAs and the predictor
//                rows of both CTAs, so each operand byte is fetched into shared memory once per pair.
//                The token rows sit as 1 KiB swizzle atoms (8 rows x 64 features) in the order (8-row group,
//                chunk): one TMA box then brings BOTH chunks of a page (the pools are described to TMA as
//                [group][chunk][row][64]), and the groups of one chunk are a uniform 2 KiB apart for the
//                operand descriptor.  A stage is one copy per page -- 8 + 1 with 16-token pages in any order
//                (an SM starts only about one copy per 80 cycles whatever its size, and a stage is ~1000
//                cycles of tensor work) -- one per run of 64 consecutive rows, or one when the CTA's 128
//                tokens lie consecutively in the pool
//   K phase    : acc0[tok, feat] (M = tokens: 128 per CTA, N = 256 features of both heads)
//                -> a thread owns (token, head): scores of the head's G query heads, tile max / exp2 /
//                   sum over the CTA's 128 tokens; the probabilities go to the CTA that owns the
//                   head in the V phase (local or distributed shared memory)
//   V phase    : acc1[feat, tok] (M = features: head r on CTA r, N = 256 tokens of both CTAs)
//                -> a thread owns (feature, half of the tokens): o = sum_tok p[tok] * acc[tok]
//   result     : one split-K partial per 128 tokens and query head.
//
// acc0 and acc1 are separate halves of tensor memory, so the K epilogue runs under the V-phase
// MMAs and the V epilogue under the next item's K-phase MMAs.  Warp roles per CTA: warps 0 and 10 TMA
// (alternate stages: with 16-token pages in no particular order a stage is up to 17 copies per CTA, and one
// warp does not issue them as fast as the tensor cores consume a stage; measured 6 % on such pools, nothing
// on consecutive pages), warp 1 MMA issue (only in the pair's first CTA) and tensor-memory allocation,
// warps 2..9 epilogue.
// Every wait is bounded; when one runs out the kernel raises the status word and winds down.
#include "recon_tc.h"

#include <cudaTypedefs.h>
#include <cuda_fp16.h>

#include "recon_common.cuh"

namespace echokv {

namespace {

constexpr int kTileTokens = 256;                     // tokens per work item (pair of CTAs)
constexpr int kCtaTokens = 128;                      // of which each CTA owns
constexpr int kChunk = 64;                           // features per swizzled sub-tile (128 bytes of bf16)
constexpr int kRowBytes = kChunk * 2;
constexpr int kStageChunks = 2;                      // 64-feature chunks per stage
constexpr int kStages = 3;
constexpr int kXBytes = kCtaTokens * kRowBytes;      // 16 KiB: token rows of one chunk
constexpr int kAtomBytes = 8 * kRowBytes;            // 1 KiB: 8 token rows of one chunk
constexpr int kGroupBytes = kStageChunks * kAtomBytes;   // 2 KiB: an 8-row group, chunk after chunk
constexpr int kWRows = 128;                          // predictor rows per CTA: one head
constexpr int kWBytes = kWRows * kRowBytes;          // 16 KiB: predictor rows of one chunk
constexpr int kStageXBytes = kStageChunks * kXBytes;  // token rows: chunk 0, chunk 1
constexpr int kStageBytes = kStageChunks * (kXBytes + kWBytes);   // then predictor rows: chunk 0, chunk 1
constexpr int kThreads = 352;                        // warps 0 and 10: TMA, 1: MMA, 2..9: epilogue
constexpr int kEpilogueThreads = 256;
constexpr int kMaxBatchPerLaunch = 256;
constexpr int kRunTokens = 64;                       // token rows of a tall box over consecutive pages
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;                        // columns of one accumulator

struct PairParams {
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
  int b0, nb;                 // batch entries [b0, b0 + nb) are handled by this launch
  int n_q_heads, n_ret_heads, n_drop_heads, n_pairs;
  int kc_anchor, kc_total;    // 64-feature chunks of the predictor input: from the anchor, in all
  int run_pages;              // pages per tall box (kRunTokens / page_tokens), 1 = no tall boxes
  int n_sink, n_window;       // sink / recent-window tokens are not predicted (masked here)
  float scale_log2e;
  RopeTable rope;             // read by the ROPE instantiations only
  const __nv_bfloat16* bk;    // bias of the K predictor or null (ROPE instantiations only: otherwise it cancels)
  float* s_out;               // KS instantiations: scores [b][query head][l_cap], base-2 units
  int l_cap;
  // KS instantiations, when set: no scores at all -- the predicted rows themselves (bias added, rotated if
  // store_rotate) are written as bf16 to store_out[b][token][store_width] at the head's flat dims
  __nv_bfloat16* store_out;
  int store_tokens, store_width, store_rotate;
  int store_half;             // the rows are written as fp16 instead of bf16 (value rows of the prefill-shaped call)
};

template <int G>
struct PairSmemTail {
  float P[2][G][kTileTokens];        // [item parity][query head][token of the tile]: this CTA's head
  float qs[2][G][128];               // queries of both heads of the pair * scale * log2e
  float kb[2][128];                  // bias of the K predictor for the pair's heads (rotating variant)
  float red_max[8][G];
  float red_sum[8][G];
  int cum_tiles[kMaxBatchPerLaunch + 1];
  unsigned long long full_bar[kStages];      // used in the first CTA: both CTAs' copies complete on it
  unsigned long long empty_bar[kStages];
  unsigned long long acc_full_bar[2];
  unsigned long long acc_empty_bar[2];       // used in the first CTA: both CTAs' epilogues arrive on it
  unsigned long long p_ready_bar;            // both CTAs' K epilogues arrive: P of an item is complete
  uint32_t tmem_base;
  int abort_flag;
};


// kind::f16: bf16 x bf16 -> fp32, both operands K-major, M = 256 over the pair, N = 256
constexpr uint32_t kIdescPair = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);


// ROPE: the predicted key rows are rotated to their positions before q . k (Section 3.2: the predictors
// produce keys prior to the rotary embedding).
// KS ("key scores only"): the K phase alone, its scores written out instead of being turned into
// probabilities; successive work items alternate between the two accumulators, so the epilogue of one item runs
// under the MMAs of the next.  Used when the V side is evaluated with absorbed predictors.
template <int G, bool ROPE, bool KS>
__global__ void __launch_bounds__(kThreads, 1)
recon_pair_kernel(const __grid_constant__ CUtensorMap tm_anchor_k, const __grid_constant__ CUtensorMap tm_anchor_v,
                  const __grid_constant__ CUtensorMap tm_local_k, const __grid_constant__ CUtensorMap tm_local_v,
                  const __grid_constant__ CUtensorMap tm_anchor_k_run, const __grid_constant__ CUtensorMap tm_anchor_v_run,
                  const __grid_constant__ CUtensorMap tm_local_k_run, const __grid_constant__ CUtensorMap tm_local_v_run,
                  const __grid_constant__ CUtensorMap tm_anchor_k_128, const __grid_constant__ CUtensorMap tm_anchor_v_128,
                  const __grid_constant__ CUtensorMap tm_local_k_128, const __grid_constant__ CUtensorMap tm_local_v_128,
                  const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
                  const PairParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  PairSmemTail<G>& t = *reinterpret_cast<PairSmemTail<G>*>(smem + kStages * kStageBytes);
  const uint32_t stage_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();          // 0: issues the MMAs; 1: its peer
  const int pair_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  volatile int* abort_flag = &t.abort_flag;

  // ---- set-up: tile counts per sequence, barriers, tensor memory --------------------------------
  for (int i = tid; i < p.nb; i += kThreads) {
    const int b = p.b0 + i;
    const int slot = p.slots ? p.slots[b] : b;
    const int len = p.lens[b];
    int tiles = 0;
    if (slot < 0 || slot >= p.max_batch) {
      if (blockIdx.x == 0) report(p.status, ECHOKV_EBADPAGE);
    } else if (len < 1 || len > p.max_pages_per_seq * p.page_tokens) {
      if (blockIdx.x == 0) report(p.status, ECHOKV_EBADLENGTH);
    } else {
      tiles = (len + kTileTokens - 1) / kTileTokens;
    }
    t.cum_tiles[i + 1] = tiles;
  }
  if (tid == 0) {
    t.cum_tiles[0] = 0;
    t.abort_flag = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&t.full_bar[s]), 2);
      mbar_init(smem_u32(&t.empty_bar[s]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&t.acc_full_bar[i]), 1);
      mbar_init(smem_u32(&t.acc_empty_bar[i]), 2);
    }
    mbar_init(smem_u32(&t.p_ready_bar), 2);
    mbar_fence_init();
  }
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int i = 0; i < p.nb; ++i) {
      acc += t.cum_tiles[i + 1];
      t.cum_tiles[i + 1] = acc;
    }
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&t.tmem_base), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = t.tmem_base;
  const int n_items = t.cum_tiles[p.nb] * p.n_pairs;
  const int boxes = kCtaTokens / p.page_tokens;             // TMA boxes (pages) of this CTA's tokens
  const uint32_t page_bytes = p.page_tokens * kRowBytes;    // of one chunk
  const uint32_t peer_abort = mapa_u32(smem_u32(&t.abort_flag), rank ^ 1u);
  // stages per phase: two chunks each.  With an odd number of chunks (a retained width that is an odd multiple
  // of 64) the last stage's second chunk lies past the end of the pool rows and of the predictor rows: TMA fills
  // both with zeros, which add nothing to the accumulators
  const int n_steps = (p.kc_total + kStageChunks - 1) / kStageChunks;
  bool gave_up = false;

  if (warp == 0 || warp == 10) {
    // =============================== TMA producers (alternate stages) ============================
    const uint32_t mine = warp == 0 ? 0u : 1u;
    uint32_t it = 0;
    bool alive = true;
    for (int item = pair_id; item < n_items && alive; item += n_clusters) {
      const ReconItem w = decode_recon_item(t.cum_tiles, item, p.n_pairs, p.nb);
      const int b = p.b0 + w.b;
      const int slot = p.slots ? p.slots[b] : b;
      const int len = p.lens[b];
      // page of box `lane` of this CTA's half of the tile, or -1 when the box holds no cached token
      int page = -1;
      if (lane < boxes) {
        const int t0 = w.tile * kTileTokens + (int)rank * kCtaTokens + lane * p.page_tokens;
        if (t0 < len) {
          page = p.table[(size_t)slot * p.max_pages_per_seq + t0 / p.page_tokens];
          if (page < 0 || page >= p.n_pages) {
            report(p.status, ECHOKV_EBADPAGE);
            page = -1;
          }
        }
      }
      const uint32_t n_valid_boxes = __popc(__ballot_sync(0xffffffffu, page >= 0));
      const uint32_t stage_tx = kStageChunks * (n_valid_boxes * page_bytes + kWBytes);
      // all of this CTA's 128 tokens cached and consecutive in the pool: one copy per stage
      const int page0 = __shfl_sync(0xffffffffu, page, 0);
      const bool run128 = __all_sync(0xffffffffu, lane >= boxes || (page >= 0 && page == page0 + lane));
      // runs of consecutive pages are fetched as one tall box
      bool run_lead = false, run_member = false;
      if (p.run_pages > 1) {
        bool consecutive = page >= 0;
        for (int k = 1; k < p.run_pages; ++k) {
          const int pk = __shfl_down_sync(0xffffffffu, page, k);
          consecutive = consecutive && pk == page + k;
        }
        const int lead = lane - lane % p.run_pages;
        const bool group_run = __shfl_sync(0xffffffffu, consecutive ? 1 : 0, lead) != 0;
        run_lead = group_run && lane == lead && lane < boxes;
        run_member = group_run && lane != lead && lane < boxes;
      }
      for (int phase = 0; phase < (KS ? 1 : 2) && alive; ++phase) {
        const CUtensorMap* m_anchor = phase == 0 ? &tm_anchor_k : &tm_anchor_v;
        const CUtensorMap* m_local = phase == 0 ? &tm_local_k : &tm_local_v;
        const CUtensorMap* m_anchor_run = phase == 0 ? &tm_anchor_k_run : &tm_anchor_v_run;
        const CUtensorMap* m_local_run = phase == 0 ? &tm_local_k_run : &tm_local_v_run;
        const CUtensorMap* m_anchor_128 = phase == 0 ? &tm_anchor_k_128 : &tm_anchor_v_128;
        const CUtensorMap* m_local_128 = phase == 0 ? &tm_local_k_128 : &tm_local_v_128;
        const CUtensorMap* m_w = phase == 0 ? &tm_wk : &tm_wv;
        for (int step = 0; step < n_steps; ++step, ++it) {
          if ((it & 1u) != mine) continue;
          const uint32_t s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          // both CTAs' copies of a stage complete on the first CTA's barrier, where the MMAs are issued
          const uint32_t full = mapa_u32(smem_u32(&t.full_bar[s]), 0u);
          bool ok = true;
          if (lane == 0) ok = mbar_wait(smem_u32(&t.empty_bar[s]), ph ^ 1u, abort_flag, p.status);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) { alive = false; break; }
          const int kc0 = step * kStageChunks;              // both chunks come from the same pool (D / 64 is even)
          const bool from_anchor = kc0 < p.kc_anchor;
          const int kx0 = from_anchor ? kc0 : kc0 - p.kc_anchor;   // chunk index inside that pool's rows
          if (lane == 0) mbar_arrive_expect_tx_cluster(full, stage_tx);
          __syncwarp();
          const uint32_t x_dst = stage_base + s * kStageBytes;
          // one box = both chunks of the rows it covers, as (group, chunk) atoms
          if (run128) {
            if (lane == 0)
              tma_load_4d_pair(x_dst, from_anchor ? m_anchor_128 : m_local_128, 0, 0, kx0, page * p.page_tokens / 8, full);
          } else if (page >= 0 && !run_member) {
            const CUtensorMap* m = run_lead ? (from_anchor ? m_anchor_run : m_local_run)
                                            : (from_anchor ? m_anchor : m_local);
            tma_load_4d_pair(x_dst + lane * kStageChunks * page_bytes, m, 0, 0, kx0, page * p.page_tokens / 8, full);
          }
          if (lane == 16)
            tma_load_3d_pair(x_dst + kStageXBytes, m_w, 0, w.pair * 2 * kWRows + (int)rank * kWRows, kc0, full);
        }
      }
    }
    gave_up = !alive;
  } else if (warp == 1) {
    // =============================== MMA issuer (first CTA of the pair) ==========================
    if (rank == 0 && lane == 0) {
      uint32_t it = 0, n = 0;
      bool alive = true;
      for (int item = pair_id; item < n_items && alive; item += n_clusters, ++n) {
        for (int phase = 0; phase < (KS ? 1 : 2) && alive; ++phase) {
          // this accumulator must have been drained by both CTAs' epilogues of its previous use
          const uint32_t acc = KS ? (n & 1u) : (uint32_t)phase;
          const uint32_t use = KS ? (n >> 1) : n;            // how often this accumulator was used before
          if (!mbar_wait_cluster(smem_u32(&t.acc_empty_bar[acc]), (use & 1u) ^ 1u, abort_flag, p.status)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint32_t d_tmem = tmem + acc * kAccCols;
          for (int step = 0; step < n_steps; ++step, ++it) {
            const uint32_t s = it % kStages;
            const uint32_t ph = (it / kStages) & 1u;
            if (!mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status)) { alive = false; break; }
            tc_fence_after();
#pragma unroll
            for (int j = 0; j < kStageChunks; ++j) {
              const uint32_t x_addr = stage_base + s * kStageBytes + j * kAtomBytes;
              const uint32_t w_addr = stage_base + s * kStageBytes + kStageXBytes + j * kWBytes;
              // K phase: A = token rows (128 per CTA), B = predictor rows (128 per CTA: 256 features).
              // V phase: A = predictor rows (head r on CTA r), B = token rows (128 per CTA: 256 tokens).
              const uint64_t x_desc = umma_desc(x_addr, kGroupBytes), w_desc = umma_desc(w_addr);
              const uint64_t a_desc = phase == 0 ? x_desc : w_desc;
              const uint64_t b_desc = phase == 0 ? w_desc : x_desc;
#pragma unroll
              for (int k16 = 0; k16 < kChunk / 16; ++k16)   // +32 bytes along K = +2 in the address field
                tc_mma_bf16_pair(d_tmem, a_desc + 2 * k16, b_desc + 2 * k16, kIdescPair,
                                 (step > 0 || j > 0 || k16 > 0) ? 1u : 0u);
            }
            tc_commit_pair(smem_u32(&t.empty_bar[s]));     // the stage is free in both CTAs
          }
          if (alive) tc_commit_pair(smem_u32(&t.acc_full_bar[acc]));
        }
      }
      gave_up = !alive;
    }
    __syncwarp();
  } else {
    // =============================== epilogue (8 warps) ========================================
    const int ew = warp - 2;                 // 0..7
    const int quarter = warp & 3;            // TMEM lane quarter this warp may read
    const int sel = ew >> 2;                 // K phase: head of the pair; V phase: half of the tokens
    const int row = quarter * 32 + lane;     // TMEM lane: token of this CTA (K phase) or feature (V phase)
    const int et = tid - 64;                 // 0..255
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
    const uint32_t acc_empty0 = mapa_u32(smem_u32(&t.acc_empty_bar[0]), 0u);
    const uint32_t acc_empty1 = mapa_u32(smem_u32(&t.acc_empty_bar[1]), 0u);
    const uint32_t p_ready_local = mapa_u32(smem_u32(&t.p_ready_bar), rank);
    const uint32_t p_ready_peer = mapa_u32(smem_u32(&t.p_ready_bar), rank ^ 1u);
    uint32_t n = 0;
    bool alive = true;
    for (int item = pair_id; item < n_items && alive; item += n_clusters, ++n) {
      const ReconItem w = decode_recon_item(t.cum_tiles, item, p.n_pairs, p.nb);
      const int b = p.b0 + w.b;
      const int len = p.lens[b];
      const int n_valid = min(kTileTokens, len - w.tile * kTileTokens);   // cached tokens in the tile
      const int kvh0 = p.n_ret_heads + w.pair * 2;           // first KV head of the pair
      const bool second = w.pair * 2 + 1 < p.n_drop_heads;   // does the pair have a second head?
      const uint32_t par = n & 1u;
      const uint32_t k_acc = KS ? (n & 1u) : 0u;             // accumulator holding this item's predicted keys
      const uint32_t k_par = KS ? ((n >> 1) & 1u) : par;
      const uint32_t k_addr = lane_addr + k_acc * kAccCols;
      // queries of the pair's query heads, pre-scaled (the previous item's K epilogue is long done)
      for (int idx = et; idx < (KS && p.store_out != nullptr ? 0 : 2 * G * 128); idx += kEpilogueThreads) {
        const int hh = idx / (G * 128), rem = idx % (G * 128);
        float v = 0.f;
        if (hh == 0 || second)
          v = __bfloat162float(p.q[((size_t)b * p.n_q_heads + (size_t)(kvh0 + hh) * G) * 128 + rem]) * p.scale_log2e;
        (&t.qs[0][0][0])[idx] = v;
      }
      if constexpr (ROPE) {
        // a bias on predicted keys is rotated with them, so it no longer cancels in the softmax
        const int hh = et >> 7, j = et & 127;
        t.kb[hh][j] = (p.bk != nullptr && (hh == 0 || second))
                          ? __bfloat162float(p.bk[(size_t)(w.pair * 2 + hh) * 128 + j]) : 0.f;
      }

      // ---------------- K phase: scores and probabilities of (token `row`, head `sel`) ----------------
      // (the vote is also the barrier that publishes the queries staged above)
      if (!epilogue_all(mbar_wait(smem_u32(&t.acc_full_bar[k_acc]), k_par, abort_flag, p.status))) { alive = false; break; }
      tc_fence_after();
      float sc[G];
#pragma unroll
      for (int gi = 0; gi < G; ++gi) sc[gi] = 0.f;
      bool stored_rows = false;
      if constexpr (KS && ROPE) {
        if (p.store_out != nullptr) {
          // the predicted rows go to memory: (token `row` of this CTA, head `sel`), 128 values as bf16
          stored_rows = true;
          const int t_row = w.tile * kTileTokens + (int)rank * kCtaTokens + row;
          const bool live = t_row < len && (sel == 0 || second);
          const bool rotate = p.store_rotate != 0 && p.rope.cs != nullptr;
          const float2* cs_row = rotate ? p.rope.cs + min(t_row, p.rope.stride - 1) : nullptr;
          __nv_bfloat16* dst = p.store_out + ((size_t)b * p.store_tokens + (live ? t_row : 0)) * p.store_width +
                               (size_t)(kvh0 + sel) * 128;
#pragma unroll 1
          for (int cb = 0; cb < 4; ++cb) {
            float lo[16], hi[16];
            tmem_ld16(k_addr + sel * 128 + cb * 16, lo);
            tmem_ld16(k_addr + sel * 128 + 64 + cb * 16, hi);
            uint32_t pl[8], ph[8];
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
              float v_lo[2], v_hi[2];
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const float k_lo = lo[j + e] + t.kb[sel][cb * 16 + j + e], k_hi = hi[j + e] + t.kb[sel][64 + cb * 16 + j + e];
                if (rotate) {
                  const float2 cw = cs_row[(size_t)(cb * 16 + j + e) * p.rope.stride];
                  v_lo[e] = k_lo * cw.x - k_hi * cw.y;
                  v_hi[e] = k_hi * cw.x + k_lo * cw.y;
                } else {
                  v_lo[e] = k_lo;
                  v_hi[e] = k_hi;
                }
              }
              if (p.store_half) {
                const __half2 a2 = __floats2half2_rn(v_lo[0], v_lo[1]), b2 = __floats2half2_rn(v_hi[0], v_hi[1]);
                pl[j / 2] = *reinterpret_cast<const uint32_t*>(&a2);
                ph[j / 2] = *reinterpret_cast<const uint32_t*>(&b2);
              } else {
                const __nv_bfloat162 a2 = __floats2bfloat162_rn(v_lo[0], v_lo[1]);
                const __nv_bfloat162 b2 = __floats2bfloat162_rn(v_hi[0], v_hi[1]);
                pl[j / 2] = *reinterpret_cast<const uint32_t*>(&a2);
                ph[j / 2] = *reinterpret_cast<const uint32_t*>(&b2);
              }
            }
            if (live) {
              uint4* d_lo = reinterpret_cast<uint4*>(dst + cb * 16);
              uint4* d_hi = reinterpret_cast<uint4*>(dst + 64 + cb * 16);
              d_lo[0] = make_uint4(pl[0], pl[1], pl[2], pl[3]);
              d_lo[1] = make_uint4(pl[4], pl[5], pl[6], pl[7]);
              d_hi[0] = make_uint4(ph[0], ph[1], ph[2], ph[3]);
              d_hi[1] = make_uint4(ph[4], ph[5], ph[6], ph[7]);
            }
          }
        }
      }
      if (stored_rows) {
        // (nothing to score)
      } else if constexpr (ROPE) {
        // this thread's row is token t_rot: features j and j + 64 of the head turn by t_rot * theta^(-2j/128)
        const int t_rot = min(w.tile * kTileTokens + (int)rank * kCtaTokens + row, p.rope.stride - 1);
        const float2* cs_row = p.rope.cs + t_rot;
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
          float2 cs[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) cs[j] = cs_row[(size_t)(cb * 16 + j) * p.rope.stride];
          float lo[16], hi[16];
          tmem_ld16(k_addr + sel * 128 + cb * 16, lo);
          tmem_ld16(k_addr + sel * 128 + 64 + cb * 16, hi);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float k_lo = lo[j] + t.kb[sel][cb * 16 + j], k_hi = hi[j] + t.kb[sel][64 + cb * 16 + j];
            const float r_lo = k_lo * cs[j].x - k_hi * cs[j].y;
            const float r_hi = k_hi * cs[j].x + k_lo * cs[j].y;
#pragma unroll
            for (int gi = 0; gi < G; ++gi)
              sc[gi] = fmaf(r_hi, t.qs[sel][gi][64 + cb * 16 + j], fmaf(r_lo, t.qs[sel][gi][cb * 16 + j], sc[gi]));
          }
        }
      } else {
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float v[32];
        tmem_ld32(k_addr + sel * 128 + c * 32, v);
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          const float4* qv = reinterpret_cast<const float4*>(&t.qs[sel][gi][c * 32]);
          float acc = sc[gi];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float4 q4 = qv[j];
            acc = fmaf(v[4 * j + 0], q4.x, acc);
            acc = fmaf(v[4 * j + 1], q4.y, acc);
            acc = fmaf(v[4 * j + 2], q4.z, acc);
            acc = fmaf(v[4 * j + 3], q4.w, acc);
          }
          sc[gi] = acc;
        }
      }
      }
      const int token = (int)rank * kCtaTokens + row;        // token of the tile
      // predicted tokens only: sink and recent-window tokens are attended from the side buffers
      const int t_seq = w.tile * kTileTokens + token;
      const bool tok_valid = t_seq >= predicted_lo(len, p.n_sink) && t_seq < predicted_hi(len, p.n_sink, p.n_window);
      if constexpr (KS) {
        tc_fence_before();
        epilogue_sync();       // every warp is done reading the accumulator (and the staged queries)
        if (et == 0) mbar_arrive_cluster(k_acc ? acc_empty1 : acc_empty0);
        // scores of every token slot of the tile; slots without a predicted token read as -inf downstream
        if (p.store_out == nullptr && t_seq < p.l_cap && (sel == 0 || second)) {
          float* dst = p.s_out + ((size_t)b * p.n_q_heads + (size_t)(kvh0 + sel) * G) * p.l_cap + t_seq;
#pragma unroll
          for (int gi = 0; gi < G; ++gi) dst[(size_t)gi * p.l_cap] = tok_valid ? sc[gi] : -INFINITY;
        }
      } else {
#pragma unroll
      for (int gi = 0; gi < G; ++gi) {
        if (!tok_valid) sc[gi] = -INFINITY;
        const float wm = warp_max(sc[gi]);
        if (lane == 0) t.red_max[ew][gi] = wm;
      }
      tc_fence_before();
      epilogue_sync();       // every warp is done reading acc0
      if (et == 0) mbar_arrive_cluster(acc_empty0);
      {
        // the probabilities go to the CTA that owns head `sel` in the V phase
        const uint32_t p_dst = mapa_u32(smem_u32(&t.P[par][0][token]), (uint32_t)sel);
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          float M = t.red_max[sel * 4][gi];
#pragma unroll
          for (int w4 = 1; w4 < 4; ++w4) M = fmaxf(M, t.red_max[sel * 4 + w4][gi]);
          // a CTA without any cached token has M = -inf: its probabilities are all zero
          const float pr = tok_valid ? exp2f(sc[gi] - M) : 0.f;
          st_cluster_f32(p_dst + gi * (kTileTokens * 4), pr);
          const float ws = warp_sum(pr);
          if (lane == 0) t.red_sum[ew][gi] = ws;
        }
      }
      epilogue_sync();       // all of this CTA's probabilities are written (here and in the peer)
      if (et == 0) {
        mbar_arrive_cluster(p_ready_local);
        mbar_arrive_cluster(p_ready_peer);
      }
      if (et < 2 * G && (int)rank * kCtaTokens < n_valid) {
        const int hh = et / G, gi = et % G;
        if (hh == 0 || second) {
          float M = t.red_max[hh * 4][gi], L = 0.f;
#pragma unroll
          for (int w4 = 1; w4 < 4; ++w4) M = fmaxf(M, t.red_max[hh * 4 + w4][gi]);
#pragma unroll
          for (int w4 = 0; w4 < 4; ++w4) L += t.red_sum[hh * 4 + w4][gi];
          const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)(kvh0 + hh) * G + gi) * p.max_parts +
                              w.tile * 2 + rank;
          p.part_ml[pidx] = make_float2(M, L);
        }
      }

      // ---------------- V phase: (feature `row` of head `rank`, token half `sel`) ----------------
      {
        const bool a_ok = mbar_wait(smem_u32(&t.acc_full_bar[1]), par, abort_flag, p.status);
        const bool p_ok = a_ok && mbar_wait_cluster(smem_u32(&t.p_ready_bar), par, abort_flag, p.status);
        if (!epilogue_all(p_ok)) { alive = false; break; }
      }
      tc_fence_after();
      const int tok0 = sel * kCtaTokens;                      // first token of this thread's half
      const bool part_live = tok0 < n_valid && (rank == 0 || second);
      float o[G];
#pragma unroll
      for (int gi = 0; gi < G; ++gi) o[gi] = 0.f;
      if (part_live) {
#pragma unroll 1
        for (int c = 0; c < kCtaTokens / 32; ++c) {
          if (tok0 + c * 32 >= n_valid) break;
          float v[32];
          tmem_ld32(lane_addr + kAccCols + tok0 + c * 32, v);
          if (tok0 + (c + 1) * 32 > n_valid) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (tok0 + c * 32 + j >= n_valid) v[j] = 0.f;     // columns that hold no cached token
          }
#pragma unroll
          for (int gi = 0; gi < G; ++gi) {
            const float4* pv = reinterpret_cast<const float4*>(&t.P[par][gi][tok0 + c * 32]);
            float acc = o[gi];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float4 p4 = pv[j];
              acc = fmaf(v[4 * j + 0], p4.x, acc);
              acc = fmaf(v[4 * j + 1], p4.y, acc);
              acc = fmaf(v[4 * j + 2], p4.z, acc);
              acc = fmaf(v[4 * j + 3], p4.w, acc);
            }
            o[gi] = acc;
          }
        }
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)(kvh0 + rank) * G + gi) * p.max_parts +
                              w.tile * 2 + sel;
          p.part_o[pidx * 128 + row] = o[gi];
        }
      }
      tc_fence_before();
      epilogue_sync();       // every warp is done reading acc1 and P[par]
      if (et == 0) mbar_arrive_cluster(acc_empty1);
      }
    }
    gave_up = !alive;
  }

  // ---- teardown ------------------------------------------------------------------------------
  if (gave_up) {
    // tell the peer, and give copies and MMAs already started ample time to land
    st_cluster_u32(peer_abort, 1u);
    const long long start = clock64();
    while (clock64() - start < 4000000ll) {
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // no CTA leaves while its peer may still reach into it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, kTmemCols);
  }
}

template <int G>
constexpr size_t pair_smem_bytes() {
  return 1024 + (size_t)kStages * kStageBytes + sizeof(PairSmemTail<G>);
}

template <int G, bool ROPE, bool KS>
cudaError_t launch_g(const TcLayerMaps& anchor, const CUtensorMap& lk, const CUtensorMap& lv, const CUtensorMap& lkr,
                     const CUtensorMap& lvr, const CUtensorMap& lk8, const CUtensorMap& lv8, const TcLayerMaps& layer,
                     const PairParams& p, int n_clusters, cudaStream_t stream) {
  const size_t smem = pair_smem_bytes<G>();
  cudaError_t e = cudaFuncSetAttribute(recon_pair_kernel<G, ROPE, KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // a persistent grid: no more CTA pairs than can be resident together (a pair shares a GPC)
  static int resident_pairs = 0;   // per instantiation
  if (resident_pairs == 0) {
    cfg.gridDim = dim3(2 * n_clusters, 1, 1);
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, recon_pair_kernel<G, ROPE, KS>, &cfg);
    if (e != cudaSuccess) return e;
    resident_pairs = n < 1 ? 1 : n;
  }
  if (n_clusters > resident_pairs) n_clusters = resident_pairs;
  cfg.gridDim = dim3(2 * n_clusters, 1, 1);
  return cudaLaunchKernelEx(&cfg, recon_pair_kernel<G, ROPE, KS>, anchor.k_grp_page, anchor.v_grp_page, lk, lv,
                            anchor.k_grp_64, anchor.v_grp_64, lkr, lvr, anchor.k_grp_128, anchor.v_grp_128, lk8, lv8,
                            layer.wk_half, layer.wv_half, p);
}

template <int G>
cudaError_t launch_g(const TcLayerMaps& anchor, const CUtensorMap& lk, const CUtensorMap& lv, const CUtensorMap& lkr,
                     const CUtensorMap& lvr, const CUtensorMap& lk8, const CUtensorMap& lv8, const TcLayerMaps& layer,
                     const PairParams& p, int n_clusters, cudaStream_t stream) {
  if (p.s_out != nullptr) {
    if (p.rope.cs == nullptr) return cudaErrorInvalidValue;     // (only built for rotated keys)
    return launch_g<G, true, true>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream);
  }
  if (p.store_out != nullptr) return cudaErrorInvalidValue;     // (rows are stored by the G = 1 instantiation, below)
  if (p.rope.cs != nullptr) return launch_g<G, true, false>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream);
  return launch_g<G, false, false>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream);
}

}  // namespace

struct StoreRows {
  __nv_bfloat16* out = nullptr;
  int tokens = 0, width = 0, rotate = 0, half = 0;
};

static cudaError_t launch_pair_impl(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                                    const TcLayerMaps& layer, int sm_count, cudaStream_t stream, float* s_out,
                                    int l_cap, const StoreRows& store = StoreRows()) {
  if (!anchor.pools_ready || !layer.weights_ready) return cudaErrorInvalidValue;
  if (r.m > 0 && !layer.pools_ready) return cudaErrorInvalidValue;
  const int g = a.n_q_heads / a.n_kv_heads;
  PairParams p;
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
  p.n_ret_heads = retained_heads(r, 128);
  p.n_drop_heads = a.n_kv_heads - p.n_ret_heads;
  p.n_pairs = (p.n_drop_heads + 1) / 2;
  p.kc_anchor = r.D / kChunk;
  p.kc_total = (r.D + r.m) / kChunk;
  p.scale_log2e = a.scale_log2e;
  p.n_sink = r.n_sink;
  p.n_window = r.n_window;
  p.rope = a.rope;
  p.bk = reinterpret_cast<const __nv_bfloat16*>(r.bk);
  p.s_out = s_out;
  p.l_cap = l_cap;
  p.store_out = store.out;
  p.store_tokens = store.tokens;
  p.store_width = store.width;
  p.store_rotate = store.rotate;
  p.store_half = store.half;
  p.run_pages = a.geom.page_tokens < kRunTokens ? kRunTokens / a.geom.page_tokens : 1;
  // with m == 0 the local maps are never used; pass the anchor's so the parameters stay valid
  const CUtensorMap& lk = r.m > 0 ? layer.k_grp_page : anchor.k_grp_page;
  const CUtensorMap& lv = r.m > 0 ? layer.v_grp_page : anchor.v_grp_page;
  const CUtensorMap& lkr = r.m > 0 ? layer.k_grp_64 : anchor.k_grp_64;
  const CUtensorMap& lvr = r.m > 0 ? layer.v_grp_64 : anchor.v_grp_64;
  const CUtensorMap& lk8 = r.m > 0 ? layer.k_grp_128 : anchor.k_grp_128;
  const CUtensorMap& lv8 = r.m > 0 ? layer.v_grp_128 : anchor.v_grp_128;
  if (p.kc_anchor % kStageChunks != 0) return cudaErrorInvalidValue;   // (a stage never straddles the two pools)
  const int tiles_cap = (r.capacity_tokens + kTileTokens - 1) / kTileTokens;
  for (int b0 = 0; b0 < a.batch; b0 += kMaxBatchPerLaunch) {
    p.b0 = b0;
    p.nb = a.batch - b0 < kMaxBatchPerLaunch ? a.batch - b0 : kMaxBatchPerLaunch;
    const long long max_items = (long long)p.nb * tiles_cap * p.n_pairs;
    const int n_clusters = (int)(max_items < sm_count / 2 ? max_items : sm_count / 2);
    cudaError_t e;
    if (store.out != nullptr) {      // rows to memory: no queries involved, one instantiation serves every group size
      e = launch_g<1, true, true>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream);
      if (e != cudaSuccess) return e;
      continue;
    }
    switch (g) {
      case 1: e = launch_g<1>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream); break;
      case 2: e = launch_g<2>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream); break;
      case 4: e = launch_g<4>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream); break;
      case 8: e = launch_g<8>(anchor, lk, lv, lkr, lvr, lk8, lv8, layer, p, n_clusters, stream); break;
      default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_recon_pair(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                              const TcLayerMaps& layer, int sm_count, cudaStream_t stream) {
  return launch_pair_impl(a, r, anchor, layer, sm_count, stream, nullptr, 0);
}

cudaError_t launch_recon_pair_key_scores(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                                         const TcLayerMaps& layer, float* scores, int l_cap, int sm_count,
                                         cudaStream_t stream) {
  if (scores == nullptr) return cudaErrorInvalidValue;
  return launch_pair_impl(a, r, anchor, layer, sm_count, stream, scores, l_cap);
}

cudaError_t launch_recon_pair_store(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                                    const TcLayerMaps& layer, bool values, __nv_bfloat16* out, int out_tokens,
                                    int out_width, int sm_count, cudaStream_t stream) {
  if (out == nullptr) return cudaErrorInvalidValue;
  StoreRows store;
  store.out = out;
  store.tokens = out_tokens;
  store.width = out_width;
  store.rotate = values ? 0 : 1;                 // (keys are rotated only if a.rope is set; values never)
  store.half = values ? 1 : 0;                   // (value rows are fp16: see the attention kernel that reads them)
  if (!values) return launch_pair_impl(a, r, anchor, layer, sm_count, stream, nullptr, 0, store);
  // the V predictor over the V pools: the same kernel with the V maps in the K places
  auto as_keys = [](const TcLayerMaps& m) {
    TcLayerMaps t = m;
    t.k_pool = m.v_pool; t.k_pool_run = m.v_pool_run; t.k_pool_run128 = m.v_pool_run128;
    t.k_grp_page = m.v_grp_page; t.k_grp_64 = m.v_grp_64; t.k_grp_128 = m.v_grp_128;
    t.wk = m.wv; t.wk_half = m.wv_half; t.wk_head = m.wv_head;
    return t;
  };
  const TcLayerMaps av = as_keys(anchor), lv = as_keys(layer);
  return launch_pair_impl(a, r, av, lv, sm_count, stream, nullptr, 0, store);
}

}  // namespace echokv
