// Pieces the two fused reconstruct-then-attend kernels (one CTA per SM; CTA pairs) share: the barrier of their
// epilogue warps, the shared-memory operand descriptor and the work-item numbering.
#pragma once

#include "ptx_sm100.cuh"

namespace echokv {

constexpr int kReconEpilogueThreads = 256;   // warps 2..9 of either kernel

__device__ __forceinline__ void epilogue_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// Barrier over the 256 epilogue threads that also ANDs a flag, so that all of them take the same
// decision after a bounded wait (a warp that left alone would strand the others at a barrier).
__device__ __forceinline__ bool epilogue_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 256, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(ok ? 1u : 0u)
      : "memory");
  return r != 0;
}

// Shared-memory matrix descriptor of a K-major bf16 operand whose rows are 128 bytes (64 features) in the
// 128-byte swizzle; 8-row groups are group_bytes apart (1024 when the rows follow one another).
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t group_bytes = 1024) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);          // start address
  d |= static_cast<uint64_t>(1) << 16;                              // leading byte offset (unused here)
  d |= static_cast<uint64_t>(group_bytes >> 4) << 32;               // stride between 8-row groups
  d |= static_cast<uint64_t>(1) << 46;                              // descriptor version of sm_100
  d |= static_cast<uint64_t>(2) << 61;                              // 128-byte swizzle
  return d;
}

// Work item -> (sequence of the launch, token tile, pair of dropped heads).  Tiles of all sequences are numbered
// consecutively (cum_tiles: exclusive prefix sums of the tiles per sequence, nb + 1 entries); items are
// token-tile-major, so that the CTAs that need the same token tile run together.
struct ReconItem {
  int b, tile, pair;
};
__device__ __forceinline__ ReconItem decode_recon_item(const int* cum_tiles, int item, int n_pairs, int nb) {
  ReconItem it;
  const int tg = item / n_pairs;
  it.pair = item - tg * n_pairs;
  int lo = 0, hi = nb;   // largest b with cum_tiles[b] <= tg
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cum_tiles[mid] <= tg) lo = mid; else hi = mid;
  }
  it.b = lo;
  it.tile = tg - cum_tiles[lo];
  return it;
}

}  // namespace echokv
