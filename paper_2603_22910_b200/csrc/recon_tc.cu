// Fused reconstruct-then-attend on the 5th-generation tensor cores (sm_100a).
//
// For every dropped KV head of a compressed layer the predictor of Eq. 3 is a dense
// contraction over D_in = D + m input features per cached token, so it runs as tcgen05.mma
// with the accumulators in tensor memory; Eq. 7 is then evaluated straight on the accumulators:
//
//   work item  = (sequence b, tile of 256 tokens, pair of dropped heads)
//   K phase    : acc[half][tok, feat] = X_K[tok, :] . W_K[feat, :]    tokens on TMEM lanes
//                -> each epilogue thread owns one token row: score = q . row (per query head of
//                   the group), tile max / exp2 / sum, probabilities go to shared memory
//   V phase    : acc[head][feat, tok] = W_V[feat, :] . X_V[tok, :]    features on TMEM lanes
//                -> each epilogue thread owns one output feature: o = sum_tok p[tok] * acc[tok]
//   result     : one split-K partial (max, sum, o) per item and query head; the merge kernel
//                combines the tiles of a sequence.
//
// Both phases stream the same shared-memory stage: 256 token rows x 64 features of the predictor
// input (one TMA box per cache page, taken through the block table, from the anchor layer's pool
// for features < D and from this layer's pool of retained dims after that) and 256 predictor rows
// x 64 features, all bf16 with the 128-byte swizzle the MMA descriptors expect.  In the K phase the
// token rows are the A operand (two M = 128 halves) and the predictor rows B (N = 256); in the V
// phase the roles swap.  The predicted K and V never leave the SM.
//
// Warp roles: warp 0 issues TMA, warp 1 issues MMA (and owns the TMEM allocation), warps 2..9 are
// the epilogue (two per TMEM lane quarter, one per accumulator half).  Every wait is bounded: when
// one runs out the kernel raises the status word, drains what it started and exits.
#include "recon_tc.h"

#include <cudaTypedefs.h>

#include "recon_common.cuh"

namespace echokv {

namespace {

constexpr int kStages = 3;
constexpr int kTileTokens = kTcPartTokens;           // 256
constexpr int kChunk = 64;                           // features per stage (128 bytes of bf16)
constexpr int kRowBytes = kChunk * 2;                // 128
constexpr int kXBytes = kTileTokens * kRowBytes;     // 32 KiB
constexpr int kWRows = 256;                          // predictor rows per stage: two heads
constexpr int kWBytes = kWRows * kRowBytes;          // 32 KiB
constexpr int kStageBytes = kXBytes + kWBytes;       // 64 KiB
constexpr int kThreads = 320;
constexpr int kEpilogueThreads = 256;
constexpr int kMaxBatchPerLaunch = 256;
constexpr int kRunTokens = 64;                       // token rows of a tall box over consecutive pages
constexpr int kTmemCols = 512;

struct TcParams {
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
  const int32_t* choose;      // null, or: run only if this device word holds choose_value (ReconArgs::choose)
  int choose_value;
};

template <int G>
struct TcSmemTail {
  float P[2 * G][kTileTokens];       // probabilities of the tile, per (head of the pair, query head)
  float qs[2][G][128];               // queries * scale * log2e
  float kb[2][128];                  // bias of the K predictor for the pair's heads (rotating variant)
  float red_max[8][2 * G];
  float red_sum[8][2 * G];
  int cum_tiles[kMaxBatchPerLaunch + 1];
  unsigned long long full_bar[kStages];
  unsigned long long empty_bar[kStages];
  unsigned long long acc_full_bar;
  unsigned long long acc_empty_bar;
  unsigned long long drain_bar;
  uint32_t tmem_base;
  int abort_flag;
};


// kind::f16 instruction: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 256
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);


// ROPE: the predicted key rows are rotated to their positions before q . k (Section 3.2: the predictors
// produce keys prior to the rotary embedding).
template <int G, bool ROPE>
__global__ void __launch_bounds__(kThreads, 1)
recon_tc_kernel(const __grid_constant__ CUtensorMap tm_anchor_k, const __grid_constant__ CUtensorMap tm_anchor_v,
                const __grid_constant__ CUtensorMap tm_local_k, const __grid_constant__ CUtensorMap tm_local_v,
                const __grid_constant__ CUtensorMap tm_anchor_k_run, const __grid_constant__ CUtensorMap tm_anchor_v_run,
                const __grid_constant__ CUtensorMap tm_local_k_run, const __grid_constant__ CUtensorMap tm_local_v_run,
                const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
                const TcParams p) {
  if (p.choose != nullptr && *p.choose != p.choose_value) return;      // (the other kernel launched for this work runs)
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  TcSmemTail<G>& t = *reinterpret_cast<TcSmemTail<G>*>(smem + kStages * kStageBytes);
  const uint32_t stage_base = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
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
      mbar_init(smem_u32(&t.full_bar[s]), 1);
      mbar_init(smem_u32(&t.empty_bar[s]), 1);
    }
    mbar_init(smem_u32(&t.acc_full_bar), 1);
    mbar_init(smem_u32(&t.acc_empty_bar), 1);
    mbar_init(smem_u32(&t.drain_bar), 1);
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
    tmem_alloc(smem_u32(&t.tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = t.tmem_base;
  const int n_items = t.cum_tiles[p.nb] * p.n_pairs;
  const int boxes = kTileTokens / p.page_tokens;            // TMA boxes (pages) per token tile
  const uint32_t page_bytes = p.page_tokens * kRowBytes;

  if (warp == 0) {
    // =============================== TMA producer ===============================================
    uint32_t it = 0;
    uint32_t issued[kStages];
#pragma unroll
    for (int s = 0; s < kStages; ++s) issued[s] = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const ReconItem w = decode_recon_item(t.cum_tiles, item, p.n_pairs, p.nb);
      const int b = p.b0 + w.b;
      const int slot = p.slots ? p.slots[b] : b;
      const int len = p.lens[b];
      // page of box `lane` of this tile, or -1 when the box holds no cached token
      int page = -1;
      if (lane < boxes) {
        const int t0 = w.tile * kTileTokens + lane * p.page_tokens;
        if (t0 < len) {
          page = p.table[(size_t)slot * p.max_pages_per_seq + t0 / p.page_tokens];
          if (page < 0 || page >= p.n_pages) {
            report(p.status, ECHOKV_EBADPAGE);
            page = -1;
          }
        }
      }
      const uint32_t n_valid_boxes = __popc(__ballot_sync(0xffffffffu, page >= 0));
      const uint32_t tx_bytes = n_valid_boxes * page_bytes + kWBytes;
      // Pages that follow one another in the pool are fetched together: when the run_pages pages of
      // an aligned group (kRunTokens token rows) are consecutive, the group's first lane issues one
      // tall box for all of them -- far fewer TMA operations than one per 16-token page.
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
        for (int kc = 0; kc < p.kc_total; ++kc, ++it) {
          const uint32_t s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          const uint32_t full = smem_u32(&t.full_bar[s]);
          bool ok = true;
          if (lane == 0) ok = mbar_wait(smem_u32(&t.empty_bar[s]), ph ^ 1u, abort_flag, p.status);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) { alive = false; break; }
          if (lane == 0) mbar_arrive_expect_tx(full, tx_bytes);
          __syncwarp();
          const uint32_t x_dst = stage_base + s * kStageBytes;
          if (page >= 0 && !run_member) {
            const bool from_anchor = kc < p.kc_anchor;
            const CUtensorMap* m = run_lead ? (from_anchor ? m_anchor_run : m_local_run)
                                            : (from_anchor ? m_anchor : m_local);
            tma_load_2d(x_dst + lane * page_bytes, m, (from_anchor ? kc : kc - p.kc_anchor) * kChunk,
                        page * p.page_tokens, full);
          }
          if (lane == 16) tma_load_2d(x_dst + kXBytes, m_w, kc * kChunk, w.pair * kWRows, full);
          issued[s] = it + 1;
        }
      }
    }
    if (!alive && lane == 0) {
      // drain: let every copy this warp started land before the CTA leaves
#pragma unroll
      for (int s = 0; s < kStages; ++s) {
        if (issued[s] == 0) continue;
        const uint32_t ph = ((issued[s] - 1) / kStages) & 1u;
        const long long start = clock64();
        while (!mbar_try_wait(smem_u32(&t.full_bar[s]), ph) && clock64() - start < kWaitLimitCycles) {
        }
      }
    }
  } else if (warp == 1) {
    // =============================== MMA issuer ================================================
    if (lane == 0) {
      uint32_t it = 0, round = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
        for (int phase = 0; phase < 2 && alive; ++phase, ++round) {
          // accumulators must have been drained by the epilogue of the previous round
          if (!mbar_wait(smem_u32(&t.acc_empty_bar), (round & 1u) ^ 1u, abort_flag, p.status)) { alive = false; break; }
          tc_fence_after();
          for (int kc = 0; kc < p.kc_total; ++kc, ++it) {
            const uint32_t s = it % kStages;
            const uint32_t ph = (it / kStages) & 1u;
            if (!mbar_wait(smem_u32(&t.full_bar[s]), ph, abort_flag, p.status)) { alive = false; break; }
            tc_fence_after();
            const uint32_t x_addr = stage_base + s * kStageBytes;
            const uint32_t w_addr = x_addr + kXBytes;
            // K phase: A = token rows (two halves of 128), B = 256 predictor rows.
            // V phase: A = predictor rows (one head of 128 each), B = 256 token rows.
            const uint32_t a_addr = phase == 0 ? x_addr : w_addr;
            const uint32_t b_addr = phase == 0 ? w_addr : x_addr;
#pragma unroll
            for (int k16 = 0; k16 < kChunk / 16; ++k16) {
              const uint64_t bd = umma_desc(b_addr + k16 * 32);
              const uint32_t acc = (kc > 0 || k16 > 0) ? 1u : 0u;
              tc_mma_bf16(tmem, umma_desc(a_addr + k16 * 32), bd, kIdesc, acc);
              tc_mma_bf16(tmem + 256, umma_desc(a_addr + 128 * kRowBytes + k16 * 32), bd, kIdesc, acc);
            }
            tc_commit(smem_u32(&t.empty_bar[s]));     // stage is free once these MMAs have read it
          }
          if (alive) tc_commit(smem_u32(&t.acc_full_bar));
        }
      }
      if (!alive) {
        // drain: wait (bounded) until every MMA issued so far has retired
        tc_commit(smem_u32(&t.drain_bar));
        const long long start = clock64();
        while (!mbar_try_wait(smem_u32(&t.drain_bar), 0) && clock64() - start < kWaitLimitCycles) {
        }
      }
    }
    __syncwarp();
  } else {
    // =============================== epilogue (8 warps) ========================================
    const int ew = warp - 2;                 // 0..7
    const int quarter = warp & 3;            // TMEM lane quarter this warp may read
    const int half = ew >> 2;                // which accumulator
    const int row = quarter * 32 + lane;     // TMEM lane: token (K phase) or feature (V phase)
    const int et = tid - 64;                 // 0..255
    const uint32_t t_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16) + half * 256;
    uint32_t round = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < n_items && alive; item += gridDim.x) {
      const ReconItem w = decode_recon_item(t.cum_tiles, item, p.n_pairs, p.nb);
      const int b = p.b0 + w.b;
      const int len = p.lens[b];
      const int n_valid = min(kTileTokens, len - w.tile * kTileTokens);
      const int kvh0 = p.n_ret_heads + w.pair * 2;           // first KV head of the pair
      const bool second = w.pair * 2 + 1 < p.n_drop_heads;   // does the pair have a second head?
      // queries of the pair's query heads, pre-scaled
      for (int idx = et; idx < 2 * G * 128; idx += kEpilogueThreads) {
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

      // ---------------- K phase: scores and probabilities ----------------
      // (the vote is also the barrier that publishes the queries staged above)
      if (!epilogue_all(mbar_wait(smem_u32(&t.acc_full_bar), round & 1u, abort_flag, p.status))) { alive = false; break; }
      tc_fence_after();
      float sc[2][G];
#pragma unroll
      for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int gi = 0; gi < G; ++gi) sc[hh][gi] = 0.f;
      if constexpr (ROPE) {
        // this thread's row is token t_rot: features j and j + 64 of a head turn by t_rot * theta^(-2j/128);
        // 16 frequencies at a time, shared by the two heads of the pair
        const int t_rot = min(w.tile * kTileTokens + half * 128 + row, p.rope.stride - 1);
        const float2* cs_row = p.rope.cs + t_rot;
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
          float2 cs[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) cs[j] = cs_row[(size_t)(cb * 16 + j) * p.rope.stride];
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            float lo[16], hi[16];
            tmem_ld16(t_addr + hh * 128 + cb * 16, lo);
            tmem_ld16(t_addr + hh * 128 + 64 + cb * 16, hi);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float k_lo = lo[j] + t.kb[hh][cb * 16 + j], k_hi = hi[j] + t.kb[hh][64 + cb * 16 + j];
              const float r_lo = k_lo * cs[j].x - k_hi * cs[j].y;
              const float r_hi = k_hi * cs[j].x + k_lo * cs[j].y;
#pragma unroll
              for (int gi = 0; gi < G; ++gi)
                sc[hh][gi] = fmaf(r_hi, t.qs[hh][gi][64 + cb * 16 + j], fmaf(r_lo, t.qs[hh][gi][cb * 16 + j], sc[hh][gi]));
            }
          }
        }
      } else {
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float v[32];
          tmem_ld32(t_addr + hh * 128 + c * 32, v);
#pragma unroll
          for (int gi = 0; gi < G; ++gi) {
            const float4* qv = reinterpret_cast<const float4*>(&t.qs[hh][gi][c * 32]);
            float acc = sc[hh][gi];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float4 q4 = qv[j];
              acc = fmaf(v[4 * j + 0], q4.x, acc);
              acc = fmaf(v[4 * j + 1], q4.y, acc);
              acc = fmaf(v[4 * j + 2], q4.z, acc);
              acc = fmaf(v[4 * j + 3], q4.w, acc);
            }
            sc[hh][gi] = acc;
          }
        }
      }
      }
      const int token = half * 128 + row;
      // predicted tokens only: sink and recent-window tokens are attended from the side buffers
      const int t_seq = w.tile * kTileTokens + token;
      const bool tok_valid = t_seq >= predicted_lo(len, p.n_sink) && t_seq < predicted_hi(len, p.n_sink, p.n_window);
#pragma unroll
      for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          if (!tok_valid) sc[hh][gi] = -INFINITY;
          const float wm = warp_max(sc[hh][gi]);
          if (lane == 0) t.red_max[ew][hh * G + gi] = wm;
        }
      epilogue_sync();
#pragma unroll
      for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
          float M = t.red_max[0][hh * G + gi];
#pragma unroll
          for (int w8 = 1; w8 < 8; ++w8) M = fmaxf(M, t.red_max[w8][hh * G + gi]);
          const float pr = tok_valid ? exp2f(sc[hh][gi] - M) : 0.f;
          t.P[hh * G + gi][token] = pr;
          const float ws = warp_sum(pr);
          if (lane == 0) t.red_sum[ew][hh * G + gi] = ws;
          sc[hh][gi] = M;
        }
      tc_fence_before();
      epilogue_sync();       // probabilities visible; every warp is done reading the accumulators
      if (et == 0) mbar_arrive(smem_u32(&t.acc_empty_bar));
      if (et < 2 * G) {
        const int hh = et / G, gi = et % G;
        if (hh == 0 || second) {
          float M = t.red_max[0][et], L = 0.f;
#pragma unroll
          for (int w8 = 1; w8 < 8; ++w8) M = fmaxf(M, t.red_max[w8][et]);
#pragma unroll
          for (int w8 = 0; w8 < 8; ++w8) L += t.red_sum[w8][et];
          const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)(kvh0 + hh) * G + gi) * p.max_parts + w.tile;
          p.part_ml[pidx] = make_float2(M, L);
        }
      }
      ++round;

      // ---------------- V phase: weighted sum of predicted V rows ----------------
      if (!epilogue_all(mbar_wait(smem_u32(&t.acc_full_bar), round & 1u, abort_flag, p.status))) { alive = false; break; }
      tc_fence_after();
      float o[G];
#pragma unroll
      for (int gi = 0; gi < G; ++gi) o[gi] = 0.f;
      if (half == 0 || second) {
#pragma unroll 1
        for (int c = 0; c < kTileTokens / 32; ++c) {
          if (c * 32 >= n_valid) break;
          float v[32];
          tmem_ld32(t_addr + c * 32, v);
          if ((c + 1) * 32 > n_valid) {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (c * 32 + j >= n_valid) v[j] = 0.f;     // columns that hold no cached token
          }
#pragma unroll
          for (int gi = 0; gi < G; ++gi) {
            const float4* pv = reinterpret_cast<const float4*>(&t.P[half * G + gi][c * 32]);
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
          const size_t pidx = ((size_t)b * p.n_q_heads + (size_t)(kvh0 + half) * G + gi) * p.max_parts + w.tile;
          p.part_o[pidx * 128 + row] = o[gi];
        }
      }
      tc_fence_before();
      epilogue_sync();
      if (et == 0) mbar_arrive(smem_u32(&t.acc_empty_bar));
      ++round;
    }
  }

  // ---- teardown ------------------------------------------------------------------------------
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
}

template <int G>
constexpr size_t tc_smem_bytes() {
  return 1024 + (size_t)kStages * kStageBytes + sizeof(TcSmemTail<G>);
}

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(sym);
  }
  return fn;
}

// bf16 matrix [rows][cols] row-major, boxes of box_rows x 64 columns, 128-byte swizzle
cudaError_t encode_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                      CUtensorMapL2promotion promo) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return cudaErrorNotSupported;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {kChunk, box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int G, bool ROPE>
cudaError_t launch_g(const CUtensorMap& ak, const CUtensorMap& av, const CUtensorMap& lk, const CUtensorMap& lv,
                     const CUtensorMap& akr, const CUtensorMap& avr, const CUtensorMap& lkr, const CUtensorMap& lvr,
                     const CUtensorMap& wk, const CUtensorMap& wv, const TcParams& p, int grid,
                     cudaStream_t stream) {
  const size_t smem = tc_smem_bytes<G>();
  cudaError_t e = cudaFuncSetAttribute(recon_tc_kernel<G, ROPE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  recon_tc_kernel<G, ROPE><<<grid, kThreads, smem, stream>>>(ak, av, lk, lv, akr, avr, lkr, lvr, wk, wv, p);
  return cudaGetLastError();
}

template <int G>
cudaError_t launch_g(const CUtensorMap& ak, const CUtensorMap& av, const CUtensorMap& lk, const CUtensorMap& lv,
                     const CUtensorMap& akr, const CUtensorMap& avr, const CUtensorMap& lkr, const CUtensorMap& lvr,
                     const CUtensorMap& wk, const CUtensorMap& wv, const TcParams& p, int grid,
                     cudaStream_t stream) {
  if (p.rope.cs != nullptr) return launch_g<G, true>(ak, av, lk, lv, akr, avr, lkr, lvr, wk, wv, p, grid, stream);
  return launch_g<G, false>(ak, av, lk, lv, akr, avr, lkr, lvr, wk, wv, p, grid, stream);
}

}  // namespace

// Exercises the give-up path of the kernels' bounded waits without putting anything in flight: one warp waits, with
// the same routine and a short limit, on a barrier that nothing ever arrives on; a second warp, as the kernels'
// other roles do, waits on a barrier of its own and must leave through the abort flag the first one raises.  No TMA
// copy is issued and no tensor memory is allocated, so nothing is pending when the block returns.
__global__ void __launch_bounds__(64) bounded_wait_probe_kernel(int32_t* status, long long limit_cycles, int* left_by) {
  __shared__ unsigned long long bars[2];
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    mbar_fence_init();
  }
  __syncthreads();
  volatile int* flag = &abort_flag;
  const int warp = threadIdx.x >> 5;
  bool ok = true;
  if ((threadIdx.x & 31) == 0) {
    // warp 0 runs out of time; warp 1 has a limit a thousand times longer and must be released by the flag
    ok = mbar_wait(smem_u32(&bars[warp]), 0, flag, status, warp == 0 ? limit_cycles : limit_cycles * 1000);
    left_by[warp] = ok ? 0 : (abort_flag ? 1 : 2);
  }
  __syncthreads();
}

cudaError_t launch_bounded_wait_probe(int32_t* status, long long limit_cycles, int* left_by, cudaStream_t stream) {
  bounded_wait_probe_kernel<<<1, 64, 0, stream>>>(status, limit_cycles, left_by);
  return cudaGetLastError();
}

bool tc_shape_supported(int dtype, int head_dim, int page_tokens, int D, int m) {
  if (dtype != ECHOKV_BF16 || head_dim != 128) return false;
  if (page_tokens != 16 && page_tokens != 32 && page_tokens != 64 && page_tokens != 128) return false;
  return D % kChunk == 0 && m % kChunk == 0 && D > m;
}

// The same matrix seen as [cols / 64][rows][64]: a box of box_chunks x box_rows x 64 lands in shared memory
// as box_chunks consecutive swizzled sub-tiles of box_rows rows, one per 64-column chunk.
cudaError_t encode_3d_chunks(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                             uint32_t box_chunks, CUtensorMapL2promotion promo) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return cudaErrorNotSupported;
  cuuint64_t dims[3] = {kChunk, rows, cols / kChunk};
  cuuint64_t strides[2] = {cols * 2, kChunk * 2};
  cuuint32_t box[3] = {kChunk, box_rows, box_chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// The same matrix seen as [rows / 8][cols / 64][8][64] (8-row groups outermost): a box of box_rows rows x 2 chunks
// lands in shared memory as 1 KiB swizzle atoms (8 rows x 64 columns) in the order (group, chunk).  A chunk past
// the last column reads as zeros.
cudaError_t encode_4d_groups(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                             CUtensorMapL2promotion promo) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return cudaErrorNotSupported;
  if (rows % 8 != 0 || box_rows % 8 != 0) return cudaErrorInvalidValue;
  cuuint64_t dims[4] = {kChunk, 8, cols / kChunk, rows / 8};
  cuuint64_t strides[3] = {cols * 2, kChunk * 2, 8 * cols * 2};
  cuuint32_t box[4] = {kChunk, 8, 2, box_rows / 8};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t encode_chunked_3d_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, int box_rows,
                                  int box_chunks) {
  return encode_3d_chunks(map, base, rows, cols, box_rows, box_chunks, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

// General form: bf16 tensor of `rank` dims (innermost first; strides in bytes for dims 1 .. rank-1), boxes in the
// 128-byte swizzle (the innermost box extent is 64 elements), out-of-range elements read as zero.
cudaError_t encode_tiled_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                              const uint64_t* strides, const uint32_t* box) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (!fn) return cudaErrorNotSupported;
  if (rank < 2 || rank > 5) return cudaErrorInvalidValue;
  cuuint64_t d[5], st[4];
  cuuint32_t bx[5], estr[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    bx[i] = box[i];
    estr[i] = 1;
    if (i + 1 < rank) st[i] = strides[i];
  }
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), d, st, bx, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t encode_pool_group_map(CUtensorMap* map, const void* pool, int width, uint64_t rows, int box_rows) {
  return encode_4d_groups(map, pool, rows, width, box_rows, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

cudaError_t encode_pool_box_map(CUtensorMap* map, const void* pool, int width, uint64_t rows, int box_rows) {
  return encode_2d(map, pool, rows, width, box_rows, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
}

cudaError_t tc_encode_pool_maps(TcLayerMaps* maps, const void* k_pool, int k_width, const void* v_pool, int v_width,
                                uint64_t rows, int page_tokens) {
  cudaError_t e;
  const CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_128B;
  if (k_width > 0) {
    if ((e = encode_2d(&maps->k_pool, k_pool, rows, k_width, page_tokens, promo)) != cudaSuccess) return e;
    // boxes of 64 token rows: runs of consecutive pages, or part of a page that is taller
    if ((e = encode_2d(&maps->k_pool_run, k_pool, rows, k_width, kRunTokens, promo)) != cudaSuccess) return e;
    // CTA-pair kernel: 128 consecutive token rows x two 64-feature chunks in one copy
    // (of a pool one chunk wide the box's second chunk lies outside the tensor and reads as zeros)
    if ((e = encode_3d_chunks(&maps->k_pool_run128, k_pool, rows, k_width, 128, 2, promo)) != cudaSuccess) return e;
    if ((e = encode_4d_groups(&maps->k_grp_page, k_pool, rows, k_width, page_tokens, promo)) != cudaSuccess) return e;
    if ((e = encode_4d_groups(&maps->k_grp_64, k_pool, rows, k_width, 64, promo)) != cudaSuccess) return e;
    if ((e = encode_4d_groups(&maps->k_grp_128, k_pool, rows, k_width, 128, promo)) != cudaSuccess) return e;
  }
  if (v_width > 0) {
    if ((e = encode_2d(&maps->v_pool, v_pool, rows, v_width, page_tokens, promo)) != cudaSuccess) return e;
    if ((e = encode_2d(&maps->v_pool_run, v_pool, rows, v_width, kRunTokens, promo)) != cudaSuccess) return e;
    if ((e = encode_3d_chunks(&maps->v_pool_run128, v_pool, rows, v_width, 128, 2, promo)) != cudaSuccess) return e;
    if ((e = encode_4d_groups(&maps->v_grp_page, v_pool, rows, v_width, page_tokens, promo)) != cudaSuccess) return e;
    if ((e = encode_4d_groups(&maps->v_grp_64, v_pool, rows, v_width, 64, promo)) != cudaSuccess) return e;
    if ((e = encode_4d_groups(&maps->v_grp_128, v_pool, rows, v_width, 128, promo)) != cudaSuccess) return e;
    // absorbed mode, V side: 64 consecutive token rows x four 64-feature chunks in one copy
    if (v_width >= 256) {
      if ((e = encode_3d_chunks(&maps->v_pool_tok64x4, v_pool, rows, v_width, 64, 4, promo)) != cudaSuccess) return e;
    }
  }
  maps->pools_ready = true;
  return cudaSuccess;
}

cudaError_t tc_encode_weight_maps(TcLayerMaps* maps, const void* Wk, const void* Wv, int d_drop, int d_in) {
  cudaError_t e;
  if (Wk != nullptr) {      // (no K predictor where the keys are kept whole)
    e = encode_2d(&maps->wk, Wk, d_drop, d_in, kWRows, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (e != cudaSuccess) return e;
    e = encode_3d_chunks(&maps->wk_half, Wk, d_drop, d_in, kWRows / 2, 2, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (e != cudaSuccess) return e;
    e = encode_2d(&maps->wk_head, Wk, d_drop, d_in, kWRows / 2, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (e != cudaSuccess) return e;
  }
  e = encode_2d(&maps->wv, Wv, d_drop, d_in, kWRows, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
  if (e != cudaSuccess) return e;
  e = encode_3d_chunks(&maps->wv_half, Wv, d_drop, d_in, kWRows / 2, 2, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
  if (e != cudaSuccess) return e;
  e = encode_2d(&maps->wv_head, Wv, d_drop, d_in, kWRows / 2, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
  if (e != cudaSuccess) return e;
  maps->weights_ready = true;
  return cudaSuccess;
}

cudaError_t launch_recon_tc(const AttnArgs& a, const ReconArgs& r, const TcLayerMaps& anchor,
                            const TcLayerMaps& layer, int sm_count, cudaStream_t stream) {
  if (!anchor.pools_ready || !layer.weights_ready) return cudaErrorInvalidValue;
  if (r.m > 0 && !layer.pools_ready) return cudaErrorInvalidValue;
  const int g = a.n_q_heads / a.n_kv_heads;
  TcParams p;
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
  p.n_pairs = (p.n_drop_heads + 1) / 2;
  p.kc_anchor = r.D / kChunk;
  p.kc_total = (r.D + r.m) / kChunk;
  p.scale_log2e = a.scale_log2e;
  p.n_sink = r.n_sink;
  p.n_window = r.n_window;
  p.rope = a.rope;
  p.bk = reinterpret_cast<const __nv_bfloat16*>(r.bk);
  p.run_pages = a.geom.page_tokens < kRunTokens ? kRunTokens / a.geom.page_tokens : 1;
  // with m == 0 the local maps are never used; pass the anchor's so the parameters stay valid
  const CUtensorMap& lk = r.m > 0 ? layer.k_pool : anchor.k_pool;
  const CUtensorMap& lv = r.m > 0 ? layer.v_pool : anchor.v_pool;
  const CUtensorMap& lkr = r.m > 0 ? layer.k_pool_run : anchor.k_pool_run;
  const CUtensorMap& lvr = r.m > 0 ? layer.v_pool_run : anchor.v_pool_run;
  const int tiles_cap = (r.capacity_tokens + kTileTokens - 1) / kTileTokens;
  for (int b0 = 0; b0 < a.batch; b0 += kMaxBatchPerLaunch) {
    p.b0 = b0;
    p.nb = a.batch - b0 < kMaxBatchPerLaunch ? a.batch - b0 : kMaxBatchPerLaunch;
    const long long max_items = (long long)p.nb * tiles_cap * p.n_pairs;
    const int grid = (int)(max_items < sm_count ? max_items : sm_count);
    cudaError_t e;
    switch (g) {
      case 1: e = launch_g<1>(anchor.k_pool, anchor.v_pool, lk, lv, anchor.k_pool_run, anchor.v_pool_run, lkr, lvr,
                                layer.wk, layer.wv, p, grid, stream); break;
      case 2: e = launch_g<2>(anchor.k_pool, anchor.v_pool, lk, lv, anchor.k_pool_run, anchor.v_pool_run, lkr, lvr,
                                layer.wk, layer.wv, p, grid, stream); break;
      case 4: e = launch_g<4>(anchor.k_pool, anchor.v_pool, lk, lv, anchor.k_pool_run, anchor.v_pool_run, lkr, lvr,
                                layer.wk, layer.wv, p, grid, stream); break;
      case 8: e = launch_g<8>(anchor.k_pool, anchor.v_pool, lk, lv, anchor.k_pool_run, anchor.v_pool_run, lkr, lvr,
                                layer.wk, layer.wv, p, grid, stream); break;
      default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace echokv
