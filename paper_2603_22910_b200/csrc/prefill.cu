// Prefill-shaped attention: the last n_q tokens of every sequence are queries at once (the paper's
// Section 5.4 notes that the dropped parts of the cache can be evicted already during the pre-filling
// phase; later chunks of a prompt then attend a compressed cache with many queries).
//
// With many queries per sequence the cache is rebuilt ONCE per call instead of once per query:
//   1. the stored dims of every cached token are gathered from the paged pool into contiguous rows
//      (gather_rows_kernel; keys rotated to their positions if a rotary table is set),
//   2. the dropped dims are predicted on the tensor cores and written beside them (Eq. 3; the
//      row-storing mode of the CTA-pair kernel),
//   3. a causal attention kernel (prefill_attn_ws_kernel: tcgen05, warp-specialised) evaluates Eq. 7 over those
//      rows, online softmax in fp32,
//   4. with sink / recent-window tokens at full precision (Section 4.1) every query is the decode step of the
//      sequence cut off at its own position: step 3 then covers the tokens the query sees as predicted (those more
//      than n_window - 1 positions before it, the sink left out), and prefill_band_kernel adds the query's own sink
//      and window tokens from their stored values and combines the two by log-sum-exp.
// The rebuilt rows are 16-bit in a caller-owned scratch, as in the paper's own materialise-then-attend
// design; the decode path never writes them.  K~ rows are bf16 (the S = Q K^T MMA takes bf16 queries).  V~ rows
// are fp16, and so are the probabilities of the P V MMA: a query that sees a handful of tokens returns nearly one
// V~ row, so the rounding of that row shows unaveraged in the output -- 2^-9 |v| in bf16, 2^-12 |v| in fp16
// (stored bf16 values are exact in fp16 between 6e-5 and 65504; probabilities stay below 2^15).
#include "prefill.h"

#include <cuda_fp16.h>

#include "ptx_sm100.cuh"
#include "recon_tc.h"

namespace echokv {

namespace {

// ---------------------------------------------------------------------------------------------
// 1. stored dims of a paged pool (rows of `width` dims) -> out[b][t][out_width] at flat dims 0 .. copy_width-1
//    (whole heads of 128)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gather_rows_kernel(const __nv_bfloat16* __restrict__ pool, int width,
                                                          int copy_width, __nv_bfloat16* __restrict__ out, int out_tokens,
                                                          int out_width, const int32_t* __restrict__ slots,
                                                          const int32_t* __restrict__ lens, PageGeom g, RopeTable rope,
                                                          int zero_tail, int block_tokens, int32_t* status, int to_half) {
  const int b = blockIdx.y, t0 = blockIdx.x * block_tokens;
  const int slot = slots ? slots[b] : b;
  const int len = lens[b];
  if (slot < 0 || slot >= g.max_batch || len < 1 || len > g.max_pages_per_seq * g.page_tokens) return;
  if (zero_tail > 0) {
    // rows len .. (next multiple of zero_tail) - 1 become zeros over the whole row: a consumer that reads whole
    // tiles of rows multiplies them by zero weights, which garbage (a NaN pattern) would not survive
    const int end = min(out_tokens, (len + zero_tail - 1) / zero_tail * zero_tail);
    const int pieces = out_width / 8;
    const bool any = t0 < end && t0 + block_tokens > len;        // (most blocks hold no such row)
    for (int it = threadIdx.x; any && it < block_tokens * pieces; it += blockDim.x) {
      const int t = t0 + it / pieces;
      if (t >= len && t < end)
        *reinterpret_cast<uint4*>(out + ((size_t)b * out_tokens + t) * (size_t)out_width + (it % pieces) * 8) =
            make_uint4(0u, 0u, 0u, 0u);
    }
  }
  if (t0 >= len || copy_width == 0) return;
  const int n_heads = copy_width / 128;
  // item = (token of the tile, head, 8-dim piece c of the head's first half, with its partner piece 64 dims on);
  // a thread takes four items at a time: four page look-ups, then eight loads, then the stores, so that they overlap
  constexpr int kBatch = 4;
  const int n_items = block_tokens * n_heads * 8;
  const int c = threadIdx.x & 7;                   // (the block size is a multiple of 8: the same for all its items)
  for (int it0 = threadIdx.x; it0 < n_items; it0 += blockDim.x * kBatch) {
    int tok[kBatch], head[kBatch], page[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int it = it0 + u * blockDim.x;
      head[u] = (it >> 3) % n_heads;
      tok[u] = it < n_items ? t0 + it / (8 * n_heads) : len;       // (len: nothing to do)
      page[u] = tok[u] < len ? g.table[(size_t)slot * g.max_pages_per_seq + tok[u] / g.page_tokens] : 0;
    }
    uint4 lo[kBatch], hi[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      if (tok[u] < len && (page[u] < 0 || page[u] >= g.n_pages)) {
        report(status, ECHOKV_EBADPAGE);
        tok[u] = len;
      }
      if (tok[u] < len) {
        const __nv_bfloat16* src = pool + ((size_t)page[u] * g.page_tokens + tok[u] % g.page_tokens) * (size_t)width +
                                   head[u] * 128 + c * 8;
        lo[u] = *reinterpret_cast<const uint4*>(src);
        hi[u] = *reinterpret_cast<const uint4*>(src + 64);
      }
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      if (tok[u] >= len) continue;
      const int t = tok[u];
      if (rope.cs != nullptr) {
        uint32_t lw[4] = {lo[u].x, lo[u].y, lo[u].z, lo[u].w}, hw[4] = {hi[u].x, hi[u].y, hi[u].z, hi[u].w};
        const float2* cs = rope.cs + min(t, rope.stride - 1);
#pragma unroll
        for (int e2 = 0; e2 < 4; ++e2) {
          float r_lo[2], r_hi[2];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const float k_lo = h ? __uint_as_float(lw[e2] & 0xffff0000u) : __uint_as_float(lw[e2] << 16);
            const float k_hi = h ? __uint_as_float(hw[e2] & 0xffff0000u) : __uint_as_float(hw[e2] << 16);
            const float2 w = cs[(size_t)(c * 8 + 2 * e2 + h) * rope.stride];
            r_lo[h] = k_lo * w.x - k_hi * w.y;
            r_hi[h] = k_hi * w.x + k_lo * w.y;
          }
          const __nv_bfloat162 a = __floats2bfloat162_rn(r_lo[0], r_lo[1]), bb = __floats2bfloat162_rn(r_hi[0], r_hi[1]);
          lw[e2] = *reinterpret_cast<const uint32_t*>(&a);
          hw[e2] = *reinterpret_cast<const uint32_t*>(&bb);
        }
        lo[u] = make_uint4(lw[0], lw[1], lw[2], lw[3]);
        hi[u] = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      } else if (to_half) {
        // the same values as fp16 (value rows; exact for every stored value a cache holds in practice)
        uint32_t lw[4] = {lo[u].x, lo[u].y, lo[u].z, lo[u].w}, hw[4] = {hi[u].x, hi[u].y, hi[u].z, hi[u].w};
#pragma unroll
        for (int e2 = 0; e2 < 4; ++e2) {
          const __half2 a = __floats2half2_rn(__uint_as_float(lw[e2] << 16), __uint_as_float(lw[e2] & 0xffff0000u));
          const __half2 bb = __floats2half2_rn(__uint_as_float(hw[e2] << 16), __uint_as_float(hw[e2] & 0xffff0000u));
          lw[e2] = *reinterpret_cast<const uint32_t*>(&a);
          hw[e2] = *reinterpret_cast<const uint32_t*>(&bb);
        }
        lo[u] = make_uint4(lw[0], lw[1], lw[2], lw[3]);
        hi[u] = make_uint4(hw[0], hw[1], hw[2], hw[3]);
      }
      __nv_bfloat16* dst = out + ((size_t)b * out_tokens + t) * (size_t)out_width + head[u] * 128 + c * 8;
      *reinterpret_cast<uint4*>(dst) = lo[u];
      *reinterpret_cast<uint4*>(dst + 64) = hi[u];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// 3. causal attention of n_q query rows over contiguous bf16 rows, on the 5th-generation tensor cores
//    (tcgen05, accumulators in tensor memory), the steps given to different warps so that they overlap
// ---------------------------------------------------------------------------------------------
constexpr int kTcTile = 128;                     // query rows per tile, keys per tile
constexpr int kTcChunkBytes = kTcTile * 128;     // [128 rows x 64 dims] bf16, 128-byte swizzle
constexpr int kTcTileBytes = 2 * kTcChunkBytes;  // 128 dims
constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// two probabilities as an fp16 pair (the A operand of the P V MMA)
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ uint64_t pf_desc_kmajor(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}
// M-major operand made of [K rows][64 M-elements] tiles in the 128-byte swizzle: 8-row groups along K are 1024 bytes
// apart, successive 64-element blocks along M are block_bytes apart
__device__ __forceinline__ uint64_t pf_desc_mmajor(uint32_t smem_addr, uint32_t block_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);
  d |= static_cast<uint64_t>(block_bytes >> 4) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// One CTA per (256 query rows, query head, sequence): two query tiles x = 0, 1 of 128 rows share every key / value tile,
// and while the tensor cores work for one of them the other one's softmax runs.  (With few queries per sequence the
// 256 rows are all the rows of 2, 4 or 8 query heads of one KV head instead.)
//   warps 0-7 / 8-15 softmax of tile 0 / 1, two threads per query row (64 keys of the tile each; four warps per
//                    scheduler, so that their special-function, ALU and FMA work overlaps).  Probabilities are taken
//                    against a reference maximum per row, 2^(s - ref): o / l does not depend on the reference, and
//                    bf16 and fp32 hold large values as precisely as small ones, so the reference only has to move
//                    before anything could overflow.  The common case is therefore taken speculatively, without
//                    looking for the maximum at all: if a thread's 64 probabilities sum to less than 2^40, nothing
//                    moves; one vote of the row's two warps confirms it.  Otherwise, and on the first and the
//                    diagonal tiles, the tile is redone the careful way (masks, maxima exchanged through shared
//                    memory, reference moved to the new maximum, O rescaled in tensor memory).  Probabilities go
//                    back as bf16 over the first 32 of the thread's own 64 columns of S.
//   warp 16          one thread issues every MMA:  S_x = Q_x K^T (A, B from shared memory, K-major) and
//                    O_x += P_x V (A = P_x from tensor memory, B = the value tile as stored [key][dim]: N-major).
//   warp 17          one thread issues the TMA loads: Q once, then key tiles (3 stages) and value tiles (2 stages).
// Tensor memory: S_0 | S_1 | O_0 | O_1, 128 columns each.  MMAs of one thread run in the order issued, so S_x(t + 1),
// issued right after O_x += P_x(t) V(t), overwrites P_x(t) only after it was read, and its completion tells the
// softmax warps that O_x is at rest as well.  Every wait on an mbarrier is bounded; the named barriers only join the
// two warps of a row pair, which take the same path through every tile (their votes also make them leave together
// when a wait ran out).
constexpr int kWsKStages = 3, kWsVStages = 2;
constexpr int kWsSoftmaxWarps = 16;
constexpr int kWsThreads = (kWsSoftmaxWarps + 2) * 32;
constexpr int kWsTailBytes = 3072;                                   // the tail sits in front of the tiles
// P V: fp16 x fp16 -> fp32 (formats 0), M = 128, N = 128, B operand N-major
constexpr uint32_t kIdescPV = (1u << 4) | ((128u >> 3) << 17) | ((128u >> 4) << 24) | (1u << 16);
constexpr float kWsGrowLog2 = 8.f;                // the careful path moves the reference if the maximum is this far above it
constexpr float kWsSumLimit = 32768.f;            // 2^15: a half-row's probabilities summing to less leave the reference
                                                  // alone (and every one of them fits fp16)

struct PfWsTail {
  float ex[2][2][kTcTile];         // [query tile][half][row]: row maxima, at the end row sums
  unsigned long long q_full;
  unsigned long long k_full[kWsKStages], k_empty[kWsKStages];
  unsigned long long v_full[kWsVStages], v_empty[kWsVStages];
  unsigned long long s_full[2], p_ready[2], o_done[2], drain;
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(PfWsTail) <= kWsTailBytes, "tail does not fit in front of the tiles");

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// barrier `id` over the 64 threads of a row pair's two warps; returns whether any of them passed a set flag
__device__ __forceinline__ bool pair_any(int id, bool flag) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %2, 0;\n\t"
      "bar.red.or.pred p, %1, 64, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(flag ? 1u : 0u)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void pair_sync(int id) { asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory"); }

__global__ void __launch_bounds__(kWsThreads, 1)
prefill_attn_ws_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, float* __restrict__ out, int n_q, int n_q_heads,
                       int n_kv_heads, const int32_t* __restrict__ slots, const int32_t* __restrict__ lens,
                       int max_batch, int capacity, float scale_log2e, int rows_per_head, int32_t* status,
                       int shift, int n_skip, float* __restrict__ lse_out) {
  // shift, n_skip: query row at position pos attends keys n_skip <= t <= pos - shift (plain causal attention: 0, 0);
  // lse_out (may be null): [B][n_q][H_q] log2 of the row's softmax denominator in the kernel's base-2 units
  // (-inf for a row that attends nothing; its output row is zero)
  // tail | Q tile 0, 1 | K stages | V stages; the tiles need 1024-byte alignment, and with all of the shared memory in
  // use there is no room to round the start up
  extern __shared__ __align__(1024) unsigned char pf_ws_raw[];
  PfWsTail& t = *reinterpret_cast<PfWsTail*>(pf_ws_raw);
  const uint32_t q_addr = smem_u32(pf_ws_raw) + kWsTailBytes, k_addr = q_addr + 2 * kTcTileBytes,
                 v_addr = k_addr + kWsKStages * kTcTileBytes;
  const int b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // The CTA's 256 query rows: rows 256 qt .. + 255 of one query head (rows_per_head = 0), or -- with few queries per
  // sequence -- rows 0 .. rows_per_head - 1 of 256 / rows_per_head query heads that share their KV head
  // (rows_per_head = 128, 64 or 32, at least n_q).  A tile whose rows all lie past n_q is not worked on at all.
  const int by = blockIdx.y, row_base = (int)blockIdx.x * 2 * kTcTile;
  const int heads_per_cta = rows_per_head ? 2 * kTcTile / rows_per_head : 1;
  // (tile x, row r of the tile) -> query head and query row
  auto head_of = [&](int x, int r) { return rows_per_head ? by * heads_per_cta + (x * kTcTile + r) / rows_per_head : by; };
  auto query_of = [&](int x, int r) { return rows_per_head ? r % rows_per_head : row_base + x * kTcTile + r; };
  const int n_act = (rows_per_head || row_base + kTcTile < n_q) ? 2 : 1;      // (tile 0 always holds a query)
  const int kvh = head_of(0, 0) / (n_q_heads / n_kv_heads);
  const int slot = slots ? slots[b] : b;
  const int len = lens[b];
  const bool misaligned = (q_addr & 1023u) != 0;
  const bool unusable = misaligned || slot < 0 || slot >= max_batch || len < n_q || len > capacity;
  const int last_row = rows_per_head ? n_q - 1 : min(n_q, row_base + n_act * kTcTile) - 1;
  const int kv_end = len - n_q + last_row + 1 - shift;      // keys this CTA's rows may see
  if (unusable || kv_end <= n_skip) {                       // (the latter: none of the rows attends anything here)
    if (unusable && tid == 0 && blockIdx.x == 0 && blockIdx.y == 0)
      report(status, misaligned ? ECHOKV_ECUDA : slot < 0 || slot >= max_batch ? ECHOKV_EBADPAGE : ECHOKV_EBADLENGTH);
    if (tid < 256) {
      const int x = tid >> 7, i = query_of(x, tid & 127);
      if (i < n_q && x < n_act) {
        const size_t row = ((size_t)b * n_q + i) * n_q_heads + head_of(x, tid & 127);
        float4* dst = reinterpret_cast<float4*>(out + row * 128);
        for (int c = 0; c < 32; ++c) dst[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lse_out != nullptr) lse_out[row] = -INFINITY;
      }
    }
    return;
  }
  volatile int* abort_flag = &t.abort_flag;
  if (tid == 0) {
    t.abort_flag = 0;
    mbar_init(smem_u32(&t.q_full), 1);
    for (int s = 0; s < kWsKStages; ++s) {
      mbar_init(smem_u32(&t.k_full[s]), 1);
      mbar_init(smem_u32(&t.k_empty[s]), 1);
    }
    for (int s = 0; s < kWsVStages; ++s) {
      mbar_init(smem_u32(&t.v_full[s]), 1);
      mbar_init(smem_u32(&t.v_empty[s]), 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(smem_u32(&t.s_full[x]), 1);
      mbar_init(smem_u32(&t.p_ready[x]), 256);
      mbar_init(smem_u32(&t.o_done[x]), 1);
    }
    mbar_init(smem_u32(&t.drain), 1);
    mbar_fence_init();
  }
  __syncthreads();
  if (warp == kWsSoftmaxWarps) {
    tmem_alloc(smem_u32(&t.tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = t.tmem_base;

  const int n_tiles = (kv_end + kTcTile - 1) / kTcTile;

  if (warp == kWsSoftmaxWarps + 1) {
    // =============================== TMA producer ===============================================
    if (lane == 0) {
      const uint32_t qb = smem_u32(&t.q_full);
      mbar_arrive_expect_tx(qb, n_act * kTcTileBytes);
      if (rows_per_head) {
        // one box per (head, 64-dim chunk): rows_per_head query rows (tm_q's box is that high and one chunk deep)
        for (int j = 0; j < heads_per_cta; ++j)
          for (int c = 0; c < 2; ++c)
            tma_load_5d(q_addr + (j * rows_per_head / kTcTile) * kTcTileBytes + c * kTcChunkBytes +
                            (j * rows_per_head % kTcTile) * 128,
                        &tm_q, 0, 0, c, by * heads_per_cta + j, b, qb);
      } else {
        for (int x = 0; x < n_act; ++x)
          tma_load_5d(q_addr + x * kTcTileBytes, &tm_q, 0, row_base + x * kTcTile, 0, by, b, qb);
      }
      bool alive = true;
      int k_issued = 0, v_issued = 0;
      for (int tile = 0; tile < n_tiles && alive; ++tile) {
        {
          const int s = tile % kWsKStages, use = tile / kWsKStages;
          if (!mbar_wait(smem_u32(&t.k_empty[s]), (use & 1) ^ 1, abort_flag, status)) { alive = false; break; }
          const uint32_t full = smem_u32(&t.k_full[s]);
          mbar_arrive_expect_tx(full, kTcTileBytes);
          tma_load_4d(k_addr + s * kTcTileBytes, &tm_k, 0, tile * kTcTile, 2 * kvh, b, full);
          k_issued = tile + 1;
        }
        {
          const int s = tile % kWsVStages, use = tile / kWsVStages;
          if (!mbar_wait(smem_u32(&t.v_empty[s]), (use & 1) ^ 1, abort_flag, status)) { alive = false; break; }
          const uint32_t full = smem_u32(&t.v_full[s]);
          mbar_arrive_expect_tx(full, kTcTileBytes);
          tma_load_4d(v_addr + s * kTcTileBytes, &tm_v, 0, tile * kTcTile, 2 * kvh, b, full);
          v_issued = tile + 1;
        }
      }
      if (!alive) {
        // let every copy that was started land before the CTA leaves
        mbar_drain(qb, 0);
        for (int i = max(0, k_issued - kWsKStages); i < k_issued; ++i)
          mbar_drain(smem_u32(&t.k_full[i % kWsKStages]), (i / kWsKStages) & 1);
        for (int i = max(0, v_issued - kWsVStages); i < v_issued; ++i)
          mbar_drain(smem_u32(&t.v_full[i % kWsVStages]), (i / kWsVStages) & 1);
      }
    }
  } else if (warp == kWsSoftmaxWarps) {
    // =============================== MMA issuer ================================================
    if (lane == 0) {
      bool alive = mbar_wait(smem_u32(&t.q_full), 0, abort_flag, status);
      auto issue_s = [&](int x, int tile) {          // S_x = Q_x K(tile)^T
        const int s = tile % kWsKStages;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint64_t a = pf_desc_kmajor(q_addr + x * kTcTileBytes + (kk >> 2) * kTcChunkBytes) + 2 * (kk & 3);
          const uint64_t bd = pf_desc_kmajor(k_addr + s * kTcTileBytes + (kk >> 2) * kTcChunkBytes) + 2 * (kk & 3);
          tc_mma_bf16(tmem + x * 128, a, bd, kIdescS, kk > 0 ? 1u : 0u);
        }
        tc_commit(smem_u32(&t.s_full[x]));
        if (x == n_act - 1) tc_commit(smem_u32(&t.k_empty[s]));
      };
      if (alive) alive = mbar_wait(smem_u32(&t.k_full[0]), 0, abort_flag, status);
      if (alive) {
        tc_fence_after();
        for (int x = 0; x < n_act; ++x) issue_s(x, 0);
      }
      for (int tile = 0; tile < n_tiles && alive; ++tile) {
        const int sv = tile % kWsVStages;
        if (!mbar_wait(smem_u32(&t.v_full[sv]), (tile / kWsVStages) & 1, abort_flag, status)) { alive = false; break; }
        const uint64_t b0 = pf_desc_mmajor(v_addr + sv * kTcTileBytes, kTcChunkBytes);
        for (int x = 0; x < n_act && alive; ++x) {
          if (!mbar_wait(smem_u32(&t.p_ready[x]), tile & 1, abort_flag, status)) { alive = false; break; }
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)     // 16 keys per MMA: 8 columns of packed probabilities (each half of the keys
                                             // at the start of its own 64 columns), 2048 bytes of value rows
            tc_mma_bf16_tmem_a(tmem + 256 + x * 128, tmem + x * 128 + 64 * (kk >> 2) + 8 * (kk & 3), b0 + 128 * kk,
                               kIdescPV, (tile > 0 || kk > 0) ? 1u : 0u);
          if (tile + 1 == n_tiles) tc_commit(smem_u32(&t.o_done[x]));
          if (x == n_act - 1) tc_commit(smem_u32(&t.v_empty[sv]));
          if (tile + 1 < n_tiles) {
            if (x == 0) {
              const int sk = (tile + 1) % kWsKStages;
              if (!mbar_wait(smem_u32(&t.k_full[sk]), ((tile + 1) / kWsKStages) & 1, abort_flag, status)) { alive = false; break; }
              tc_fence_after();
            }
            issue_s(x, tile + 1);
          }
        }
      }
      if (!alive) {
        // every MMA issued so far retires before the tensor memory is given back
        tc_commit(smem_u32(&t.drain));
        mbar_drain(smem_u32(&t.drain), 0);
      }
    }
  } else if ((warp >> 3) < n_act) {
    // =============================== softmax: two threads per query row, 64 keys each ===================
    const int x = warp >> 3, hf = (warp >> 2) & 1, row = (warp & 3) * 32 + lane;
    const int pair_id = 1 + x * 4 + (warp & 3);             // named barrier of this row's two warps
    const int h = head_of(x, row);
    const int i_row = query_of(x, row);
    const bool row_ok = i_row < n_q;
    const int pos = len - n_q + i_row - shift;              // last key this query row attends here
    const uint32_t lane_base = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
    const uint32_t s_addr = lane_base + x * 128 + hf * 64, o_addr = lane_base + 256 + x * 128 + hf * 64;
    float m_ref = -INFINITY, l_run = 0.f;                   // m_ref is the same in both threads of a row
    bool alive = true;
    for (int tile = 0; tile < n_tiles; ++tile) {
      const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&t.s_full[x]), tile & 1, abort_flag, status) ? 1 : 0) != 0;
      // keys of this thread's half the row sees: the first n_vis
      const int n_vis = row_ok ? max(0, min(64, pos - (tile * kTcTile + hf * 64) + 1)) : 0;
      const int n_lo = max(0, min(64, n_skip - (tile * kTcTile + hf * 64)));    // ... but not the first n_lo
      uint32_t sr[2][32];
      float mx = -INFINITY, psum = 0.f;
      if (ok) {
        tc_fence_after();
        tmem_ld32_issue(s_addr, sr[0]);
        tmem_ld32_issue(s_addr + 32, sr[1]);
        tmem_ld_wait();
        // Speculation: every key visible and the reference where it is.  Two scores per instruction where the pipe
        // has a two-wide form (scale-and-shift, row sum).  (Measured and dropped: a cubic on the FMA pipe for part of
        // the 2^x, +10 % time at a quarter of them; looking for the row maximum beside the 2^x, +5 %.)
        const uint64_t sc2 = pack_f2(scale_log2e, scale_log2e), nm2 = pack_f2(-m_ref, -m_ref);
        uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          // 32 keys -> 16 columns of packed bf16 pairs; sr[c] is dead afterwards, so the pairs overwrite its first half
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const uint64_t x2 = fma_f2(pack_u2(sr[c][j], sr[c][j + 1]), sc2, nm2);
            float x0, x1;
            unpack_f2(x2, x0, x1);
            const float p0 = ex2_approx(x0), p1 = ex2_approx(x1);
            sum2[(j >> 1) & 1] = add_f2(sum2[(j >> 1) & 1], pack_f2(p0, p1));
            sr[c][j >> 1] = pack2(p0, p1);
          }
        }
        float a0, a1, b0, b1;
        unpack_f2(sum2[0], a0, a1);
        unpack_f2(sum2[1], b0, b1);
        psum = (a0 + a1) + (b0 + b1);
      }
      const bool careful = !ok || tile == 0 || n_vis != 64 || n_lo != 0 || !(psum < kWsSumLimit);
      if (pair_any(pair_id, careful)) {
        if (pair_any(pair_id, !ok)) { alive = false; break; }     // both warps of the row leave together
        // ---- the careful way: masks, the row maximum over both halves, O rescaled if the reference moves
        tmem_ld32_issue(s_addr, sr[0]);
        tmem_ld32_issue(s_addr + 32, sr[1]);
        tmem_ld_wait();
        mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (32 * c + j < n_vis && 32 * c + j >= n_lo) mx = fmaxf(mx, __uint_as_float(sr[c][j]));
        mx *= scale_log2e;
        t.ex[x][hf][row] = mx;
        pair_sync(pair_id);
        mx = fmaxf(mx, t.ex[x][hf ^ 1][row]);
        const bool grow = mx > m_ref + kWsGrowLog2;
        float alpha = 1.f;
        if (grow) {
          alpha = ex2_approx(m_ref - mx);      // 0 on the first tile
          m_ref = mx;
          l_run *= alpha;
        }
        if (tile > 0 && __any_sync(0xffffffffu, grow)) {
          // O_x is at rest (the MMA that wrote S came after every earlier one): rescale this thread's half of its row
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            uint32_t orow[32];
            tmem_ld32_issue(o_addr + 32 * c, orow);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) orow[j] = __float_as_uint(__uint_as_float(orow[j]) * alpha);
            tmem_st32(o_addr + 32 * c, orow);
          }
        }
        // (the scores are read once more rather than kept in registers across the rescaling)
        tmem_ld32_issue(s_addr, sr[0]);
        tmem_ld32_issue(s_addr + 32, sr[1]);
        tmem_ld_wait();
        psum = 0.f;
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const bool v0 = 32 * c + j < n_vis && 32 * c + j >= n_lo, v1 = 32 * c + j + 1 < n_vis && 32 * c + j + 1 >= n_lo;
            const float p0 = v0 ? ex2_approx(fmaf(__uint_as_float(sr[c][j]), scale_log2e, -m_ref)) : 0.f;
            const float p1 = v1 ? ex2_approx(fmaf(__uint_as_float(sr[c][j + 1]), scale_log2e, -m_ref)) : 0.f;
            psum += p0 + p1;
            sr[c][j >> 1] = pack2(p0, p1);
          }
      }
      l_run += psum;
      tmem_st16(s_addr, sr[0]);            // the packed pairs sit in the first 16 registers of each block of 32
      tmem_st16(s_addr + 16, sr[1]);
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(smem_u32(&t.p_ready[x]));
    }
    if (alive) {
      // the row's sum over both halves; every wait from here on is on the same barrier for both warps of a row
      t.ex[x][hf][row] = l_run;
      pair_sync(pair_id);
      l_run += t.ex[x][hf ^ 1][row];
      if (mbar_wait(smem_u32(&t.o_done[x]), 0, abort_flag, status)) {
        tc_fence_after();
        const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
        if (lse_out != nullptr && row_ok && hf == 0)
          lse_out[((size_t)b * n_q + i_row) * n_q_heads + h] = l_run > 0.f ? m_ref + log2f(l_run) : -INFINITY;
        float4* dst = reinterpret_cast<float4*>(out + (((size_t)b * n_q + (row_ok ? i_row : 0)) * n_q_heads + h) * 128 + hf * 64);
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          float v[32];
          tmem_ld32(o_addr + 32 * c, v);
          if (row_ok) {
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4)
              dst[8 * c + j4] = make_float4(v[4 * j4] * inv, v[4 * j4 + 1] * inv, v[4 * j4 + 2] * inv, v[4 * j4 + 3] * inv);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kWsSoftmaxWarps) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---------------------------------------------------------------------------------------------
// 4. the sink and window tokens of every query, at full precision (Section 4.1), combined with step 3
// ---------------------------------------------------------------------------------------------
// One block per (QB consecutive queries, KV head, sequence).  The query at position p reads as stored: the sink
// tokens t < min(n_sink, p + 1) -- their retained dims from the layer's pools, the rest from the side buffers -- and
// the window tokens max(n_sink, p - n_window + 1) .. p, whole rows of k_recent / v_recent.  Consecutive queries share
// all but one of these tokens, so the block reads the union once (n_sink + n_window + QB - 1 rows) and masks per
// query.  Scores: thread per token, the key row (rotated to its position if a table is set) against the QB x G query
// rows held in shared memory.  Softmax: warp per (query, head).  Values: 32 threads x 4 output dims per token, the
// block's five warps on every fifth token, summed through shared memory; then the log-sum-exp combination with what
// step 3 left in out / lse for the tokens the query sees as predicted.
constexpr int kBandThreads = 160;
constexpr int kBandSlices = kBandThreads / 32;

template <int G, int QB>
__global__ void __launch_bounds__(kBandThreads) prefill_band_kernel(AttnArgs a, PrefillBand w, int n_q,
                                                                    float* __restrict__ out,
                                                                    const float* __restrict__ lse) {
  extern __shared__ __align__(16) float band_smem[];
  constexpr int DH = 128;
  constexpr int R = QB * G;                    // (query, head) rows of the block
  using T = __nv_bfloat16;
  const int i0 = blockIdx.x * QB, kvh = blockIdx.y, b = blockIdx.z, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nq_blk = min(QB, n_q - i0);        // queries of this block
  const int n_list = w.n_sink + w.n_window;
  const int NT = n_list + QB - 1;              // most tokens the block can see
  float* qs = band_smem;                       // [R][DH], scaled
  float* sc = qs + R * DH;                     // [R][NT]: scores, then probabilities
  float* osum = sc + R * NT;                   // [R][DH]: weighted values, summed over the slices
  __shared__ float s_m[R], s_l[R];
  const int slot = a.slots ? a.slots[b] : b;
  const int len = a.lens[b];
  if (slot < 0 || slot >= a.geom.max_batch || len < n_q || len > a.geom.max_pages_per_seq * a.geom.page_tokens)
    return;                                    // (reported, and zeros written, by step 3)
  const int p_first = len - n_q + i0, p_last = p_first + nq_blk - 1;      // positions of the block's queries
  const int n_sink_u = min(w.n_sink, p_last + 1);
  const int wlo = max(w.n_sink, p_first - w.n_window + 1);
  const int n_tok = n_sink_u + max(0, p_last - wlo + 1);
  const int n_stored_k = min(max(w.mk - kvh * DH, 0), DH), n_stored_v = min(max(w.m - kvh * DH, 0), DH);
  const int n_rows = n_q + w.n_window - 1;     // rows of k_recent / v_recent per sequence; row 0 is position t_base
  const int t_base = len - n_rows;
  {
    const T* q = reinterpret_cast<const T*>(a.q) + (((size_t)b * n_q + i0) * a.n_q_heads + (size_t)kvh * G) * DH;
    for (int idx = tid; idx < R * DH; idx += kBandThreads) {
      const int qi = idx / (G * DH), rest = idx - qi * G * DH;
      qs[idx] = qi < nq_blk ? __bfloat162float(q[(size_t)qi * a.n_q_heads * DH + rest]) * a.scale_log2e : 0.f;
    }
  }
  __syncthreads();
  const T* k_pool = reinterpret_cast<const T*>(w.k_pool);
  const T* v_pool = reinterpret_cast<const T*>(w.v_pool);
  const T* k_side = reinterpret_cast<const T*>(w.k_side);
  const T* v_side = reinterpret_cast<const T*>(w.v_side);
  const T* k_recent = reinterpret_cast<const T*>(w.k_recent);
  const T* v_recent = reinterpret_cast<const T*>(w.v_recent);
  const int32_t* table = a.geom.table + (size_t)slot * a.geom.max_pages_per_seq;
  // pool row (in token rows) of sink token t
  auto pool_row = [&](int t) -> size_t {
    int page = table[t / a.geom.page_tokens];
    if (page < 0 || page >= a.geom.n_pages) {
      report(a.status, ECHOKV_EBADPAGE);
      page = 0;
    }
    return (size_t)page * a.geom.page_tokens + t % a.geom.page_tokens;
  };
  const size_t side_base = (size_t)slot * n_list;
  // ---- scores: one token per thread, against all R query rows ----
  for (int idx = tid; idx < n_tok; idx += kBandThreads) {
    const bool sink = idx < n_sink_u;
    const int t = sink ? idx : wlo + (idx - n_sink_u);
    const T* a_ptr;      // dims [0, n_a) of the head
    const T* b_ptr;      // the rest
    int n_a;
    if (sink) {
      const size_t r = n_stored_k > 0 ? pool_row(t) : 0;
      a_ptr = k_pool + r * (size_t)w.mk + (size_t)kvh * DH;
      n_a = n_stored_k;
      b_ptr = k_side + (side_base + t) * (size_t)w.d_drop + (kvh * DH + n_stored_k - w.mk);
    } else {
      a_ptr = k_recent + ((size_t)b * n_rows + (t - t_base)) * (size_t)w.D + (size_t)kvh * DH;
      n_a = DH;
      b_ptr = a_ptr;
    }
    auto k_at = [&](int j) -> const T* { return j < n_a ? a_ptr + j : b_ptr + (j - n_a); };
    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.f;
    // eight dims of the key (kv) against the same dims of every query row
    auto dot8 = [&](const float (&kv)[8], int j) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const float4 q0 = *reinterpret_cast<const float4*>(qs + r * DH + j);
        const float4 q1 = *reinterpret_cast<const float4*>(qs + r * DH + j + 4);
        acc[r] = fmaf(kv[0], q0.x, fmaf(kv[1], q0.y, fmaf(kv[2], q0.z, fmaf(kv[3], q0.w, acc[r]))));
        acc[r] = fmaf(kv[4], q1.x, fmaf(kv[5], q1.y, fmaf(kv[6], q1.z, fmaf(kv[7], q1.w, acc[r]))));
      }
    };
    if (a.rope.cs != nullptr) {
      const float2* cs = a.rope.cs + min(t, a.rope.stride - 1);
      for (int j = 0; j < DH / 2; j += 8) {
        float k_lo[8], k_hi[8], r_lo[8], r_hi[8];
        Vec16<T>::load(k_at(j), k_lo);
        Vec16<T>::load(k_at(DH / 2 + j), k_hi);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float2 cw = cs[(size_t)(j + e) * a.rope.stride];
          r_lo[e] = k_lo[e] * cw.x - k_hi[e] * cw.y;
          r_hi[e] = k_hi[e] * cw.x + k_lo[e] * cw.y;
        }
        dot8(r_lo, j);
        dot8(r_hi, DH / 2 + j);
      }
    } else {
      for (int j = 0; j < DH; j += 8) {
        float kv[8];
        Vec16<T>::load(k_at(j), kv);
        dot8(kv, j);
      }
    }
#pragma unroll
    for (int qi = 0; qi < QB; ++qi) {
      // does query qi see token t as stored?  (its sink tokens, its window)
      const int pq = p_first + qi;
      const bool seen = qi < nq_blk && (sink ? t < min(w.n_sink, pq + 1) : (t <= pq && t > pq - w.n_window));
#pragma unroll
      for (int gi = 0; gi < G; ++gi) sc[(qi * G + gi) * NT + idx] = seen ? acc[qi * G + gi] : -INFINITY;
    }
  }
  __syncthreads();
  // ---- softmax: a warp per (query, head) row ----
  for (int r = warp; r < R; r += kBandSlices) {
    float* row = sc + r * NT;
    float mx = -INFINITY;
    for (int idx = lane; idx < n_tok; idx += 32) mx = fmaxf(mx, row[idx]);
    mx = warp_max(mx);
    float l = 0.f;
    for (int idx = lane; idx < n_tok; idx += 32) {
      const float pv = mx > -INFINITY ? exp2f(row[idx] - mx) : 0.f;      // (a row of a query past the chunk: nothing)
      row[idx] = pv;
      l += pv;
    }
    l = warp_sum(l);
    if (lane == 0) {
      s_m[r] = mx;
      s_l[r] = l;
    }
  }
  for (int idx = tid; idx < R * DH; idx += kBandThreads) osum[idx] = 0.f;
  __syncthreads();
  // ---- weighted values: output dims 4 lane .. 4 lane + 3 of the head, this warp on every fifth token ----
  float o[R][4];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[r][e] = 0.f;
  auto add_token = [&](int idx, const float (&vv)[4]) {
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const float pv = sc[r * NT + idx];
#pragma unroll
      for (int e = 0; e < 4; ++e) o[r][e] = fmaf(pv, vv[e], o[r][e]);
    }
  };
  for (int idx = warp; idx < n_sink_u; idx += kBandSlices) {            // sink tokens: pool + side buffers
    float vv[4];
    const size_t prow = n_stored_v > 0 ? pool_row(idx) : 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int dim = 4 * lane + e;
      vv[e] = dim < n_stored_v
                  ? __bfloat162float(v_pool[prow * (size_t)w.m + (size_t)kvh * DH + dim])
                  : __bfloat162float(v_side[(side_base + idx) * (size_t)w.d_drop + (kvh * DH + dim - w.m)]);
    }
    add_token(idx, vv);
  }
  {
    // window tokens: rows of v_recent, four loads in flight at a time
    const int n_win = n_tok - n_sink_u;
    const T* v_col = v_recent + ((size_t)b * n_rows + (wlo - t_base)) * (size_t)w.D + (size_t)kvh * DH + 4 * lane;
    for (int i = warp; i < n_win; i += 4 * kBandSlices) {
      uint2 raw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int iu = i + u * kBandSlices;
        raw[u] = iu < n_win ? *reinterpret_cast<const uint2*>(v_col + (size_t)iu * w.D) : make_uint2(0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int iu = i + u * kBandSlices;
        if (iu < n_win) {
          const float vv[4] = {__uint_as_float(raw[u].x << 16), __uint_as_float(raw[u].x & 0xffff0000u),
                               __uint_as_float(raw[u].y << 16), __uint_as_float(raw[u].y & 0xffff0000u)};
          add_token(n_sink_u + iu, vv);
        }
      }
    }
  }
  // the slices' sums, one slice after the other
  for (int s = 0; s < kBandSlices; ++s) {
    if (warp == s) {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        float4* dst = reinterpret_cast<float4*>(osum + r * DH + 4 * lane);
        float4 v = *dst;
        v.x += o[r][0]; v.y += o[r][1]; v.z += o[r][2]; v.w += o[r][3];
        *dst = v;
      }
    }
    __syncthreads();
  }
  // ---- the combination with the predicted tokens' result ----
  for (int idx = tid; idx < nq_blk * G * DH; idx += kBandThreads) {
    const int r = idx / DH, d = idx - r * DH, qi = r / G, gi = r - qi * G;
    const size_t orow = ((size_t)b * n_q + i0 + qi) * a.n_q_heads + (size_t)kvh * G + gi;
    const float lse_a = lse[orow];                       // -inf: the query sees no token as predicted
    const float M = fmaxf(lse_a, s_m[r]);
    const float w_a = lse_a > -INFINITY ? exp2f(lse_a - M) : 0.f;
    const float w_b = exp2f(s_m[r] - M);
    const float denom = w_a + w_b * s_l[r];
    out[orow * DH + d] = (w_a * out[orow * DH + d] + w_b * osum[r * DH + d]) / denom;
  }
}

}  // namespace

cudaError_t launch_gather_rows(const AttnArgs& a, const void* pool, int width, int copy_width, __nv_bfloat16* out,
                               int out_tokens, int out_width, bool rotate, int zero_tail, cudaStream_t stream,
                               bool to_half) {
  if (copy_width == 0 && zero_tail == 0) return cudaSuccess;
  if (copy_width % 128 != 0 || copy_width > width || out_width % 8 != 0) return cudaErrorInvalidValue;
  // enough tokens per block that every thread has four items to overlap
  const int block_tokens = copy_width <= 256 ? 64 : 32;
  dim3 grid((out_tokens + block_tokens - 1) / block_tokens, a.batch);
  gather_rows_kernel<<<grid, 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(pool), width, copy_width, out, out_tokens,
                                               out_width, a.slots, a.lens, a.geom, rotate ? a.rope : RopeTable(), zero_tail,
                                               block_tokens, a.status, to_half ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t launch_prefill_attn(const AttnArgs& a, const __nv_bfloat16* k_rows, const __nv_bfloat16* v_rows,
                                int kv_tokens, int kv_width, int n_q, float* out, cudaStream_t stream, int shift,
                                int n_skip, float* lse_out) {
  if (kv_width % 64 != 0 || reinterpret_cast<uintptr_t>(a.q) % 16 != 0) return cudaErrorInvalidValue;
  CUtensorMap tm_q, tm_k, tm_v;
  // few queries per sequence: the CTA's 256 rows are 2, 4 or 8 query heads of one KV head, rows_per_head rows each
  const int group = a.n_q_heads / a.n_kv_heads;
  int rows_per_head = 0;
  for (int r = 32; r <= kTcTile; r *= 2)
    if (rows_per_head == 0 && n_q <= r && group % (2 * kTcTile / r) == 0) rows_per_head = r;
  {
    // q [B][n_q][H_q][128] seen as [B][H_q][2 chunks][n_q][64]: a box is the two 64-dim chunks of 128 query rows,
    // or one chunk of rows_per_head rows
    const uint64_t dims[5] = {64, (uint64_t)n_q, 2, (uint64_t)a.n_q_heads, (uint64_t)a.batch};
    const uint64_t strides[4] = {(uint64_t)a.n_q_heads * 256, 128, 256, (uint64_t)n_q * a.n_q_heads * 256};
    const uint32_t box[5] = {64, (uint32_t)(rows_per_head ? rows_per_head : kTcTile), rows_per_head ? 1u : 2u, 1, 1};
    const cudaError_t e = encode_tiled_bf16(&tm_q, a.q, 5, dims, strides, box);
    if (e != cudaSuccess) return e;
  }
  for (int kind = 0; kind < 2; ++kind) {
    // rows [B][kv_tokens][kv_width] seen as [B][kv_width / 64][kv_tokens][64]: a box is one head (two chunks) of 128 rows
    const uint64_t dims[4] = {64, (uint64_t)kv_tokens, (uint64_t)kv_width / 64, (uint64_t)a.batch};
    const uint64_t strides[3] = {(uint64_t)kv_width * 2, 128, (uint64_t)kv_tokens * kv_width * 2};
    const uint32_t box[4] = {64, (uint32_t)kTcTile, 2, 1};
    const cudaError_t e = encode_tiled_bf16(kind ? &tm_v : &tm_k, kind ? v_rows : k_rows, 4, dims, strides, box);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(rows_per_head ? 1 : (n_q + 2 * kTcTile - 1) / (2 * kTcTile),
            rows_per_head ? a.n_q_heads / (2 * kTcTile / rows_per_head) : a.n_q_heads, a.batch);
  const size_t smem = kWsTailBytes + (size_t)(2 + kWsKStages + kWsVStages) * kTcTileBytes;
  const cudaError_t e = cudaFuncSetAttribute(prefill_attn_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
  if (e != cudaSuccess) return e;
  prefill_attn_ws_kernel<<<grid, kWsThreads, smem, stream>>>(tm_q, tm_k, tm_v, out, n_q, a.n_q_heads, a.n_kv_heads,
                                                             a.slots, a.lens, a.geom.max_batch,
                                                             a.geom.max_pages_per_seq * a.geom.page_tokens,
                                                             a.scale_log2e, rows_per_head, a.status, shift, n_skip,
                                                             lse_out);
  return cudaGetLastError();
}

namespace {
size_t band_smem_bytes(int rows, int n_list, int qb) {
  return (size_t)(2 * rows * 128 + rows * (n_list + qb - 1)) * sizeof(float);
}
template <int G, int QB>
cudaError_t launch_band_g(const AttnArgs& a, const PrefillBand& band, int n_q, float* out, const float* lse,
                          cudaStream_t stream) {
  const size_t smem = band_smem_bytes(G * QB, band.n_sink + band.n_window, QB);
  cudaError_t e = cudaFuncSetAttribute(prefill_band_kernel<G, QB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((n_q + QB - 1) / QB, a.n_kv_heads, a.batch);
  prefill_band_kernel<G, QB><<<grid, kBandThreads, smem, stream>>>(a, band, n_q, out, lse);
  return cudaGetLastError();
}
template <int G>
cudaError_t launch_band_q(const AttnArgs& a, const PrefillBand& band, int n_q, float* out, const float* lse,
                          cudaStream_t stream) {
  // four queries per block share their tokens; a very long window (its probabilities no longer fit in shared
  // memory four queries at a time) goes one query per block
  constexpr int kQB = G >= 8 ? 2 : 4;
  if (band_smem_bytes(G * kQB, band.n_sink + band.n_window, kQB) <= 96 * 1024)
    return launch_band_g<G, kQB>(a, band, n_q, out, lse, stream);
  return launch_band_g<G, 1>(a, band, n_q, out, lse, stream);
}
}  // namespace

cudaError_t launch_prefill_band(const AttnArgs& a, const PrefillBand& band, int n_q, float* out, const float* lse,
                                cudaStream_t stream) {
  switch (a.n_q_heads / a.n_kv_heads) {
    case 1: return launch_band_q<1>(a, band, n_q, out, lse, stream);
    case 2: return launch_band_q<2>(a, band, n_q, out, lse, stream);
    case 4: return launch_band_q<4>(a, band, n_q, out, lse, stream);
    case 8: return launch_band_q<8>(a, band, n_q, out, lse, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace echokv
