// Shared declarations of the EchoKV CUDA library: status codes seen by device code,
// the split-K partial layout, and small device helpers.  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/echokv.h"

namespace echokv {

constexpr int kSimtTileTokens = 64;   // token tile of the CUDA-core reconstruct kernel
constexpr int kTcPartTokens = 256;    // tokens per work item / partial of the tcgen05 kernel
constexpr int kMaxGroup = 8;          // largest n_q_heads / n_kv_heads the kernels unroll for
constexpr float kLog2e = 1.4426950408889634f;

// Split-K partial results (Eq. 7 evaluated over one token range, in base-2 exponent units):
//   ml[(b * H_q + h) * max_parts + p] = (max score * log2e, sum of 2^(score - max))
//   o [((b * H_q + h) * max_parts + p) * d + j] = sum_t 2^(score_t - max) * V[t][j]
struct Partials {
  float2* ml;
  float* o;
  int max_parts;
};

// Geometry of one paged pool set, by value into kernels.
struct PageGeom {
  const int32_t* table;   // [max_batch][max_pages_per_seq]
  int max_batch;
  int max_pages_per_seq;
  int page_tokens;
  long long n_pages;
};

// Rotary position embedding applied when the cache is read (Section 3.2: the predictors, hence the
// cache, hold keys prior to RoPE).  cs[j * stride + t] = (cos, sin)(t * theta^(-2 j / d)) for the d/2
// frequency indices j and positions t < stride; feature j pairs with feature j + d/2.  cs == null: off.
// The same angles factored as position = 16 u + r:  coarse[u * (d/2) + j] = (cos, sin)(16 u * w_j) for
// u < stride / 16 and fine[r * (d/2) + j] = (cos, sin)(r * w_j) for r < 16 (the stored-head kernel multiplies
// the two: a 64-token stage then needs 2 KiB of table instead of 32 KiB).
struct RopeTable {
  const float2* cs = nullptr;
  int stride = 0;
  const float2* coarse = nullptr;
  const float2* fine = nullptr;
};
constexpr int kRopeFineRows = 16;

__device__ __forceinline__ void report(int32_t* status, int code) {
  // keep the first error; 0 means "none yet"
  atomicCAS(status, 0, code);
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// 16-byte global load of stored elements, widened to fp32.
template <typename T>
struct Vec16;
template <>
struct Vec16<float> {
  static constexpr int N = 4;
  __device__ __forceinline__ static void load(const float* p, float* out) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ __forceinline__ static void load(const __nv_bfloat16* p, float* out) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// two fp32 values in one 64-bit register, for the two-wide fp32 instructions of sm_100
__device__ __forceinline__ uint64_t pack_u2(uint32_t lo, uint32_t hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "r"(lo), "r"(hi));
  return v;
}
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi) { return pack_u2(__float_as_uint(lo), __float_as_uint(hi)); }
__device__ __forceinline__ void unpack_u2(uint64_t v, uint32_t& lo, uint32_t& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v));
}
__device__ __forceinline__ void unpack_f2(uint64_t v, float& lo, float& hi) {
  uint32_t a, b;
  unpack_u2(v, a, b);
  lo = __uint_as_float(a);
  hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t fma_f2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul_f2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// Resolve (sequence slot, length) of batch entry b; reports and returns false when unusable.
__device__ __forceinline__ bool resolve_sequence(const int32_t* slots, const int32_t* lens, int b,
                                                 const PageGeom& g, int32_t* status, int& slot,
                                                 int& len) {
  slot = slots ? slots[b] : b;
  len = lens[b];
  if (slot < 0 || slot >= g.max_batch) {
    report(status, ECHOKV_EBADPAGE);
    return false;
  }
  if (len < 1 || len > g.max_pages_per_seq * g.page_tokens) {
    report(status, ECHOKV_EBADLENGTH);
    return false;
  }
  return true;
}

}  // namespace echokv
