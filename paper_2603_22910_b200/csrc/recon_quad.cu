// Fused reconstruct-then-attend on CTA pairs, four dropped heads per work item (tcgen05 cta_group::2, sm_100a).
//
// The same computation as recon_pair.cu (Eq. 3 on the tensor cores, Eq. 7 on the accumulators), with the tile
// doubled along the predictor rows so that a token tile is staged once per FOUR heads:
//
//   work item  = (sequence b, tile of 256 tokens, quad of dropped heads 4q .. 4q + 3), one per CTA pair;
//                CTA r of the pair owns tokens [128 r, 128 r + 128) of the tile and heads 4q + r and 4q + r + 2
//   stage      = one 64-feature chunk: per CTA 128 token rows (16 KiB, one TMA box per page) and the 2 x 128
//                predictor rows of its two heads (32 KiB); 48 KiB, 4 deep.  Against the one-CTA kernel a stage
//                holds the same tensor work (~1100 cycles) for three quarters of the bytes and half the token-row
//                copies -- the number of copies an SM can start is what bounds that kernel on pools of small pages
//                in a random order
//   K phase    : acc[tok, feat]: two M = 256, N = 256 MMAs per 16 features (heads 4q, 4q + 1 -> columns 0..255,
//                heads 4q + 2, 4q + 3 -> columns 256..511) -> a thread owns (token, heads c and c + 2):
//                scores, tile max / exp2 / sum over the CTA's 128 tokens; the probabilities go to the CTA that owns
//                the head in the V phase (local or distributed shared memory)
//   V phase    : acc[feat, tok]: heads 4q + r (columns 0..255 = the tile's tokens) and 4q + r + 2 (columns 256..511)
//                on CTA r -> a thread owns (feature, half of the tokens) of both: o = sum_tok p[tok] * acc[tok]
//   result     : one split-K partial per 128 tokens and query head, as the pair kernel writes them.
//
// All 512 tensor-memory columns belong to the running phase, so the epilogues do not overlap the MMAs: the kernel
// is for long contractions with few query heads per KV head (G <= 2), where an epilogue is a percent or two of a
// phase.  Warp roles per CTA: warps 0 and 10 TMA (stage 0 / stage 1), warp 1 MMA issue (first CTA of the pair)
// and tensor-memory allocation, warps 2..9 epilogue.  Every wait is bounded.
#include "recon_tc.h"

#include <cudaTypedefs.h>

#include "recon_common.cuh"

namespace echokv {

namespace {

constexpr int kTileTokens = 256;                     // tokens per work item (pair of CTAs)
constexpr int kCtaTokens = 128;                      // of which each CTA owns
constexpr int kChunk = 64;                           // features per swizzled sub-tile (128 bytes of bf16)
constexpr int kRowBytes = kChunk * 2;
constexpr int kStages = 4;
constexpr int kXBytes = kCtaTokens * kRowBytes;      // 16 KiB: the CTA's token rows of one chunk
constexpr int kWRows = 128;                          // predictor rows of one head
constexpr int kWHeadBytes = kWRows * kRowBytes;      // 16 KiB: one head's rows of one chunk
constexpr int kStageBytes = kXBytes + 2 * kWHeadBytes;           // 48 KiB
constexpr int kThreads = 352;                        // warps 0 and 10: TMA, 1: MMA, 2..9: epilogue
constexpr int kMaxBatchPerLaunch = 256;
constexpr int kRunTokens = 64;                       // token rows of a tall box over consecutive pages
constexpr int kTmemCols = 512;

struct QuadParams {
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
  int n_q_heads, n_ret_heads, n_drop_heads, n_quads;
  int kc_anchor, kc_total;    // 64-feature chunks of the predictor input: from the anchor, in all
  int run_pages;              // pages per tall box (kRunTokens / page_tokens), 1 = no tall boxes
  int n_sink, n_window;       // sink / recent-window tokens are not predicted (masked here)
  float scale_log2e;
  RopeTable rope;             // read by the ROPE instantiations only
  const __nv_bfloat16* bk;    // bias of the K predictor or null (ROPE instantiations only: otherwise it cancels)
  const int32_t* choose;      // null, or: run only if this device word holds choose_value (ReconArgs::choose)
  int choose_value;
};

template <int G>
struct QuadSmemTail {
  float P[2][G][kTileTokens];        // [head slot: this CTA's heads 4q + r, 4q + r + 2][query head][token of the tile]
  float qs[4][G][128];               // queries of the quad's heads * scale * log2e
  float kb[4][128];                  // bias of the K predictor for the quad's heads (rotating variant)
  float red_max[8][2][G];            // [epilogue warp][head slot of the thread][query head]
  float red_sum[8][2][G];
  int cum_tiles[kMaxBatchPerLaunch + 1];
  unsigned long long full_bar[kStages];      // used in the first CTA: both CTAs' copies complete on it
  unsigned long long empty_bar[kStages];
  unsigned long long acc_full_bar;
  unsigned long long acc_empty_bar;          // used in the first CTA: both CTAs' epilogues arrive on it
  unsigned long long p_ready_bar;            // both CTAs' K epilogues arrive: P of an item is complete
  uint32_t tmem_base;
  int abort_flag;
};

// kind::f16: bf16 x bf16 -> fp32, both operands K-major, M = 256 over the pair, N = 256
constexpr uint32_t kIdescPair = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);

// ROPE: the predicted key rows are rotated to their positions before q . k (Section 3.2: the predictors
// produce keys prior to the rotary embedding).
template <int G, bool ROPE>
__global__ void __launch_bounds__(kThreads, 1)
recon_quad_kernel(const __grid_constant__ CUtensorMap tm_anchor_k, const __grid_constant__ CUtensorMap tm_anchor_v,
                  const __grid_constant__ CUtensorMap tm_local_k, const __grid_constant__ CUtensorMap tm_local_v,
                  const __grid_constant__ CUtensorMap tm_anchor_k_run, const __grid_constant__ CUtensorMap tm_anchor_v_run,
                  const __grid_constant__ CUtensorMap tm_local_k_run, const __grid_constant__ CUtensorMap tm_local_v_run,
                  const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
                  const QuadParams p) {
  if (p.choose != nullptr && *p.choose != p.choose_value) return;      // (both CTAs of the pair alike: the other
                                                                       // kernel launched for this work runs)
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  QuadSmemTail<G>& t = *reinterpret_cast<QuadSmemTail<G>*>(smem + kStages * kStageBytes);
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
    mbar_init(smem_u32(&t.acc_full_bar), 1);
    mbar_init(smem_u32(&t.acc_empty_bar), 2);
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
  const int n_items = t.cum_tiles[p.nb] * p.n_quads;
  const int boxes = kCtaTokens / p.page_tokens;             // TMA boxes (pages) of this CTA's tokens
  const uint32_t page_bytes = p.page_tokens * kRowBytes;    // of one chunk
  const uint32_t peer_abort = mapa_u32(smem_u32(&t.abort_flag), rank ^ 1u);
  const int n_steps = p.kc_total;                           // stages per phase: one chunk each
  bool gave_up = false;

  if (warp == 0 || warp == 10) {
    // =============================== TMA producers (alternate stages) ============================
    const uint32_t mine = warp == 0 ? 0u : 1u;
    uint32_t it = 0;
    bool alive = true;
    for (int item = pair_id; item < n_items && alive; item += n_clusters) {
      const ReconItem w = decode_recon_item(t.cum_tiles, item, p.n_quads, p.nb);
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
      const uint32_t stage_tx = n_valid_boxes * page_bytes + 2 * kWHeadBytes;
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
      for (int phase = 0; phase < 2 && alive; ++phase) {
        const CUtensorMap* m_anchor = phase == 0 ? &tm_anchor_k : &tm_anchor_v;
        const CUtensorMap* m_local = phase == 0 ? &tm_local_k : &tm_local_v;
        const CUtensorMap* m_anchor_run = phase == 0 ? &tm_anchor_k_run : &tm_anchor_v_run;
        const CUtensorMap* m_local_run = phase == 0 ? &tm_local_k_run : &tm_local_v_run;
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
          const int kc0 = step;
          const bool from_anchor = kc0 < p.kc_anchor;
          const int kx0 = from_anchor ? kc0 : kc0 - p.kc_anchor;   // chunk index inside that pool's rows
          if (lane == 0) mbar_arrive_expect_tx_cluster(full, stage_tx);
          __syncwarp();
          const uint32_t x_dst = stage_base + s * kStageBytes;
          if (run128) {
            // the CTA's 128 tokens lie consecutively in the pool: two boxes of 64 rows
            if (lane < 2)
              tma_load_2d_pair(x_dst + lane * (kRunTokens * kRowBytes), from_anchor ? m_anchor_run : m_local_run,
                               kx0 * kChunk, page0 * p.page_tokens + lane * kRunTokens, full);
          } else if (page >= 0 && !run_member) {
            const CUtensorMap* m = run_lead ? (from_anchor ? m_anchor_run : m_local_run)
                                            : (from_anchor ? m_anchor : m_local);
            tma_load_2d_pair(x_dst + lane * page_bytes, m, kx0 * kChunk, page * p.page_tokens, full);
          }
          // the predictor rows of this CTA's two heads (rows past the last dropped head read as zeros)
          if (lane == 16 || lane == 17) {
            const int k = lane - 16;
            tma_load_2d_pair(x_dst + kXBytes + k * kWHeadBytes, m_w, kc0 * kChunk,
                             (w.pair * 4 + (int)rank + 2 * k) * kWRows, full);
          }
        }
      }
    }
    gave_up = !alive;
  } else if (warp == 1) {
    // =============================== MMA issuer (first CTA of the pair) ==========================
    if (rank == 0 && lane == 0) {
      uint32_t it = 0, use = 0;
      bool alive = true;
      for (int item = pair_id; item < n_items && alive; item += n_clusters) {
        for (int phase = 0; phase < 2 && alive; ++phase, ++use) {
          // the accumulators must have been drained by both CTAs' epilogues of the previous phase
          if (!mbar_wait_cluster(smem_u32(&t.acc_empty_bar), (use & 1u) ^ 1u, abort_flag, p.status)) {
            alive = false;
            break;
          }
          tc_fence_after();
          for (int step = 0; step < n_steps; ++step, ++it) {
            const uint32_t s = it % kStages;
            const uint32_t ph = (it / kStages) & 1u;
            if (!mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status)) { alive = false; break; }
            tc_fence_after();
            {
              const uint32_t x_addr = stage_base + s * kStageBytes;
              const uint32_t w_addr = x_addr + kXBytes;
              // K phase: A = token rows (128 per CTA), B = predictor rows of one head per CTA (256 features);
              // V phase: A = predictor rows (one head per CTA), B = token rows (128 per CTA: 256 tokens).
              // Twice: heads 4q + {0, 1} into columns 0..255, heads 4q + {2, 3} into columns 256..511.
              const uint64_t x_desc = umma_desc(x_addr);
              const uint64_t w_desc0 = umma_desc(w_addr), w_desc1 = umma_desc(w_addr + kWHeadBytes);
#pragma unroll
              for (int k16 = 0; k16 < kChunk / 16; ++k16) {   // +32 bytes along K = +2 in the address field
                const uint32_t accum = (step > 0 || k16 > 0) ? 1u : 0u;
                if (phase == 0) {
                  tc_mma_bf16_pair(tmem, x_desc + 2 * k16, w_desc0 + 2 * k16, kIdescPair, accum);
                  tc_mma_bf16_pair(tmem + 256, x_desc + 2 * k16, w_desc1 + 2 * k16, kIdescPair, accum);
                } else {
                  tc_mma_bf16_pair(tmem, w_desc0 + 2 * k16, x_desc + 2 * k16, kIdescPair, accum);
                  tc_mma_bf16_pair(tmem + 256, w_desc1 + 2 * k16, x_desc + 2 * k16, kIdescPair, accum);
                }
              }
            }
            tc_commit_pair(smem_u32(&t.empty_bar[s]));     // the stage is free in both CTAs
          }
          if (alive) tc_commit_pair(smem_u32(&t.acc_full_bar));
        }
      }
      gave_up = !alive;
    }
    __syncwarp();
  } else {
    // =============================== epilogue (8 warps) ========================================
    const int ew = warp - 2;                 // 0..7
    const int quarter = warp & 3;            // TMEM lane quarter this warp may read
    const int sel = ew >> 2;                 // K phase: heads sel and sel + 2 of the quad; V phase: half of the tokens
    const int row = quarter * 32 + lane;     // TMEM lane: token of this CTA (K phase) or feature (V phase)
    const int et = tid - 64;                 // 0..255
    const uint32_t lane_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
    const uint32_t acc_empty = mapa_u32(smem_u32(&t.acc_empty_bar), 0u);
    const uint32_t p_ready_local = mapa_u32(smem_u32(&t.p_ready_bar), rank);
    const uint32_t p_ready_peer = mapa_u32(smem_u32(&t.p_ready_bar), rank ^ 1u);
    uint32_t n = 0;
    bool alive = true;
    for (int item = pair_id; item < n_items && alive; item += n_clusters, ++n) {
      const ReconItem w = decode_recon_item(t.cum_tiles, item, p.n_quads, p.nb);
      const int b = p.b0 + w.b;
      const int len = p.lens[b];
      const int n_valid = min(kTileTokens, len - w.tile * kTileTokens);   // cached tokens in the tile
      const int kvh0 = p.n_ret_heads + w.pair * 4;           // first KV head of the quad
      const int n_live = min(4, p.n_drop_heads - w.pair * 4);  // heads the quad really has
      const uint32_t par = n & 1u;
      // queries of the quad's query heads, pre-scaled (the previous item's K epilogue is long done)
      for (int idx = et; idx < 4 * G * 128; idx += 256) {
        const int c = idx / (G * 128), rem = idx % (G * 128);
        float v = 0.f;
        if (c < n_live)
          v = __bfloat162float(p.q[((size_t)b * p.n_q_heads + (size_t)(kvh0 + c) * G) * 128 + rem]) * p.scale_log2e;
        (&t.qs[0][0][0])[idx] = v;
      }
      if constexpr (ROPE) {
        // a bias on predicted keys is rotated with them, so it no longer cancels in the softmax
        for (int idx = et; idx < 4 * 128; idx += 256) {
          const int c = idx >> 7, j = idx & 127;
          t.kb[c][j] = (p.bk != nullptr && c < n_live) ? __bfloat162float(p.bk[(size_t)(w.pair * 4 + c) * 128 + j]) : 0.f;
        }
      }

      // ---------------- K phase: scores and probabilities of (token `row`, heads sel and sel + 2) ----------------
      // (the vote is also the barrier that publishes the queries staged above)
      if (!epilogue_all(mbar_wait(smem_u32(&t.acc_full_bar), 0u, abort_flag, p.status))) { alive = false; break; }
      tc_fence_after();
      float sc[2][G];
#pragma unroll
      for (int k = 0; k < 2; ++k)
#pragma unroll
        for (int gi = 0; gi < G; ++gi) sc[k][gi] = 0.f;
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int c = sel + 2 * k;             // column block of the accumulators = head of the quad
        if constexpr (ROPE) {
          // this thread's row is token t_rot: features j and j + 64 of the head turn by t_rot * theta^(-2j/128)
          const int t_rot = min(w.tile * kTileTokens + (int)rank * kCtaTokens + row, p.rope.stride - 1);
          const float2* cs_row = p.rope.cs + t_rot;
#pragma unroll 1
          for (int cb = 0; cb < 4; ++cb) {
            float2 cs[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) cs[j] = cs_row[(size_t)(cb * 16 + j) * p.rope.stride];
            float lo[16], hi[16];
            tmem_ld16(lane_addr + c * 128 + cb * 16, lo);
            tmem_ld16(lane_addr + c * 128 + 64 + cb * 16, hi);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float k_lo = lo[j] + t.kb[c][cb * 16 + j], k_hi = hi[j] + t.kb[c][64 + cb * 16 + j];
              const float r_lo = k_lo * cs[j].x - k_hi * cs[j].y;
              const float r_hi = k_hi * cs[j].x + k_lo * cs[j].y;
#pragma unroll
              for (int gi = 0; gi < G; ++gi)
                sc[k][gi] = fmaf(r_hi, t.qs[c][gi][64 + cb * 16 + j], fmaf(r_lo, t.qs[c][gi][cb * 16 + j], sc[k][gi]));
            }
          }
        } else {
#pragma unroll 1
          for (int c4 = 0; c4 < 4; ++c4) {
            float v[32];
            tmem_ld32(lane_addr + c * 128 + c4 * 32, v);
#pragma unroll
            for (int gi = 0; gi < G; ++gi) {
              const float4* qv = reinterpret_cast<const float4*>(&t.qs[c][gi][c4 * 32]);
              float acc = sc[k][gi];
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float4 q4 = qv[j];
                acc = fmaf(v[4 * j + 0], q4.x, acc);
                acc = fmaf(v[4 * j + 1], q4.y, acc);
                acc = fmaf(v[4 * j + 2], q4.z, acc);
                acc = fmaf(v[4 * j + 3], q4.w, acc);
              }
              sc[k][gi] = acc;
            }
          }
        }
      }
      const int token = (int)rank * kCtaTokens + row;        // token of the tile
      // predicted tokens only: sink and recent-window tokens are attended from the side buffers
      const int t_seq = w.tile * kTileTokens + token;
      const bool tok_valid = t_seq >= predicted_lo(len, p.n_sink) && t_seq < predicted_hi(len, p.n_sink, p.n_window);
#pragma unroll
      for (int k = 0; k < 2; ++k)
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          if (!tok_valid) sc[k][gi] = -INFINITY;
          const float wm = warp_max(sc[k][gi]);
          if (lane == 0) t.red_max[ew][k][gi] = wm;
        }
      tc_fence_before();
      epilogue_sync();       // every warp is done reading the accumulators
      if (et == 0) mbar_arrive_cluster(acc_empty);
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        // the probabilities go to the CTA that owns head sel + 2k in the V phase: CTA `sel`, head slot k
        const uint32_t p_dst = mapa_u32(smem_u32(&t.P[k][0][token]), (uint32_t)sel);
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          float M = t.red_max[sel * 4][k][gi];
#pragma unroll
          for (int w4 = 1; w4 < 4; ++w4) M = fmaxf(M, t.red_max[sel * 4 + w4][k][gi]);
          // a CTA without any cached token has M = -inf: its probabilities are all zero
          const float pr = tok_valid ? exp2f(sc[k][gi] - M) : 0.f;
          st_cluster_f32(p_dst + gi * (kTileTokens * 4), pr);
          const float ws = warp_sum(pr);
          if (lane == 0) t.red_sum[ew][k][gi] = ws;
        }
      }
      epilogue_sync();       // all of this CTA's probabilities are written (here and in the peer)
      if (et == 0) {
        mbar_arrive_cluster(p_ready_local);
        mbar_arrive_cluster(p_ready_peer);
      }
      if (et < 4 * G && (int)rank * kCtaTokens < n_valid) {
        const int c = et / G, gi = et % G;     // head of the quad, query head of its group
        if (c < n_live) {
          const int s_c = c & 1, k_c = c >> 1;   // the epilogue warps and the slot that handled head c
          float M = t.red_max[s_c * 4][k_c][gi], L = 0.f;
#pragma unroll
          for (int w4 = 1; w4 < 4; ++w4) M = fmaxf(M, t.red_max[s_c * 4 + w4][k_c][gi]);
#pragma unroll
          for (int w4 = 0; w4 < 4; ++w4) L += t.red_sum[s_c * 4 + w4][k_c][gi];
          const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)(kvh0 + c) * G + gi) * p.max_parts +
                              w.tile * 2 + rank;
          p.part_ml[pidx] = make_float2(M, L);
        }
      }

      // ---------------- V phase: (feature `row` of heads rank and rank + 2, token half `sel`) ----------------
      {
        const bool a_ok = mbar_wait(smem_u32(&t.acc_full_bar), 1u, abort_flag, p.status);
        const bool p_ok = a_ok && mbar_wait_cluster(smem_u32(&t.p_ready_bar), par, abort_flag, p.status);
        if (!epilogue_all(p_ok)) { alive = false; break; }
      }
      tc_fence_after();
      const int tok0 = sel * kCtaTokens;                      // first token of this thread's half
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int c = (int)rank + 2 * k;                      // head of the quad this CTA holds in slot k
        if (!(tok0 < n_valid && c < n_live)) continue;
        float o[G];
#pragma unroll
        for (int gi = 0; gi < G; ++gi) o[gi] = 0.f;
#pragma unroll 1
        for (int c32 = 0; c32 < kCtaTokens / 32; ++c32) {
          if (tok0 + c32 * 32 >= n_valid) break;
          float v[32];
          tmem_ld32(lane_addr + k * 256 + tok0 + c32 * 32, v);
          if (tok0 + (c32 + 1) * 32 > n_valid) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (tok0 + c32 * 32 + j >= n_valid) v[j] = 0.f;     // columns that hold no cached token
          }
#pragma unroll
          for (int gi = 0; gi < G; ++gi) {
            const float4* pv = reinterpret_cast<const float4*>(&t.P[k][gi][tok0 + c32 * 32]);
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
          const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)(kvh0 + c) * G + gi) * p.max_parts +
                              w.tile * 2 + sel;
          p.part_o[pidx * 128 + row] = o[gi];
        }
      }
      tc_fence_before();
      epilogue_sync();       // every warp is done reading the accumulators and P
      if (et == 0) mbar_arrive_cluster(acc_empty);
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
constexpr size_t quad_smem_bytes() {
  return 1024 + (size_t)kStages * kStageBytes + sizeof(QuadSmemTail<G>);
}

template <int G, bool ROPE>
cudaError_t launch_g(const TcLayerMaps& anchor, const TcLayerMaps& local, const TcLayerMaps& layer,
                     const QuadParams& p, int n_clusters, cudaStream_t stream) {
  const size_t smem = quad_smem_bytes<G>();
  cudaError_t e = cudaFuncSetAttribute(recon_quad_kernel<G, ROPE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
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
    e = cudaOccupancyMaxActiveClusters(&n, recon_quad_kernel<G, ROPE>, &cfg);
    if (e != cudaSuccess) return e;
    resident_pairs = n < 1 ? 1 : n;
  }
  if (n_clusters > resident_pairs) n_clusters = resident_pairs;
  cfg.gridDim = dim3(2 * n_clusters, 1, 1);
  return cudaLaunchKernelEx(&cfg, recon_quad_kernel<G, ROPE>, anchor.k_pool, anchor.v_pool, local.k_pool,
                            local.v_pool, anchor.k_pool_run, anchor.v_pool_run, local.k_pool_run, local.v_pool_run,
                            layer.wk_head, layer.wv_head, p);
}

}  // namespace

bool recon_quad_supported(int group) { return group == 1 || group == 2; }

cudaError_t launch_recon_quad(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                              const TcLayerMaps& layer, int sm_count, cudaStream_t stream) {
  if (!anchor.pools_ready || !layer.weights_ready) return cudaErrorInvalidValue;
  if (r.m > 0 && !layer.pools_ready) return cudaErrorInvalidValue;
  const int g = a.n_q_heads / a.n_kv_heads;
  if (!recon_quad_supported(g)) return cudaErrorInvalidValue;
  QuadParams p;
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
  p.choose = r.choose;
  p.choose_value = r.choose_value;
  p.n_q_heads = a.n_q_heads;
  p.n_ret_heads = retained_heads(r, 128);
  p.n_drop_heads = a.n_kv_heads - p.n_ret_heads;
  p.n_quads = (p.n_drop_heads + 3) / 4;
  p.kc_anchor = r.D / kChunk;
  p.kc_total = (r.D + r.m) / kChunk;
  p.scale_log2e = a.scale_log2e;
  p.n_sink = r.n_sink;
  p.n_window = r.n_window;
  p.rope = a.rope;
  p.bk = reinterpret_cast<const __nv_bfloat16*>(r.bk);
  p.run_pages = a.geom.page_tokens < kRunTokens ? kRunTokens / a.geom.page_tokens : 1;
  // with m == 0 the local maps are never used; pass the anchor's so the parameters stay valid
  const TcLayerMaps& local = r.m > 0 ? layer : anchor;
  const int tiles_cap = (r.capacity_tokens + kTileTokens - 1) / kTileTokens;
  for (int b0 = 0; b0 < a.batch; b0 += kMaxBatchPerLaunch) {
    p.b0 = b0;
    p.nb = a.batch - b0 < kMaxBatchPerLaunch ? a.batch - b0 : kMaxBatchPerLaunch;
    const long long max_items = (long long)p.nb * tiles_cap * p.n_quads;
    const int n_clusters = (int)(max_items < sm_count / 2 ? max_items : sm_count / 2);
    cudaError_t e;
    if (g == 1) {
      e = p.rope.cs != nullptr ? launch_g<1, true>(anchor, local, layer, p, n_clusters, stream)
                               : launch_g<1, false>(anchor, local, layer, p, n_clusters, stream);
    } else {
      e = p.rope.cs != nullptr ? launch_g<2, true>(anchor, local, layer, p, n_clusters, stream)
                               : launch_g<2, false>(anchor, local, layer, p, n_clusters, stream);
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace echokv
