// CUDA-core kernels of the EchoKV decode path: cache append, attention over stored heads
// (anchor layers, retained heads), the fp32-FFMA reconstruct-then-attend kernel that serves the
// fp32 test mode and shapes the tensor-core kernel does not take, and the split-K merge.
#include "kernels.h"

namespace echokv {

// ---------------------------------------------------------------------------------------------
// Rotary table (Section 3.2: keys are cached un-rotated and rotated to their position when read)
// ---------------------------------------------------------------------------------------------
// out[i] = (cos, sin)(pos * theta^(-2 j / d)); layout 0: i = j * n_pos + pos (positions 0 .. n_pos-1);
// layout 1: i = u * (d/2) + j with pos = pos_step * u.
__global__ void __launch_bounds__(256) rope_table_kernel(float2* __restrict__ out, long long n, int n_pos,
                                                         int head_dim, double theta, int layout, int pos_step) {
  const int half = head_dim / 2;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
    int j, pos;
    if (layout == 0) { j = (int)(i / n_pos); pos = (int)(i % n_pos); }
    else { j = (int)(i % half); pos = (int)(i / half) * pos_step; }
    const double angle = (double)pos * pow(theta, -2.0 * (double)j / (double)head_dim);
    double sn, cs;
    sincos(angle, &sn, &cs);
    out[i] = make_float2((float)cs, (float)sn);
  }
}

size_t rope_table_pairs(int stride, int head_dim) {
  const size_t half = head_dim / 2;
  return half * stride + (size_t)(stride / kRopeFineRows) * half + (size_t)kRopeFineRows * half;
}

RopeTable rope_table_view(const float2* buffer, int stride, int head_dim) {
  const size_t half = head_dim / 2;
  RopeTable t;
  t.cs = buffer;
  t.stride = stride;
  t.coarse = buffer + half * stride;
  t.fine = t.coarse + (size_t)(stride / kRopeFineRows) * half;
  return t;
}

cudaError_t launch_rope_table(float2* buffer, int stride, int head_dim, double theta, cudaStream_t stream) {
  const RopeTable t = rope_table_view(buffer, stride, head_dim);
  const long long half = head_dim / 2;
  const long long n[3] = {half * stride, (long long)(stride / kRopeFineRows) * half, (long long)kRopeFineRows * half};
  float2* dst[3] = {buffer, const_cast<float2*>(t.coarse), const_cast<float2*>(t.fine)};
  const int layout[3] = {0, 1, 1}, step[3] = {1, kRopeFineRows, 1};
  for (int k = 0; k < 3; ++k) {
    if (n[k] == 0) continue;
    long long blocks = (n[k] + 255) / 256;
    if (blocks > 4096) blocks = 4096;
    rope_table_kernel<<<(int)blocks, 256, 0, stream>>>(dst[k], n[k], stride, head_dim, theta, layout[k], step[k]);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// ---------------------------------------------------------------------------------------------
// Append (Section 3.1: the dropped dims of a compressed layer are simply not written; Eq. 2)
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) append_kernel(T* __restrict__ k_pool, T* __restrict__ v_pool,
                                                     int k_width, int v_width, int D, const T* __restrict__ k_new,
                                                     const T* __restrict__ v_new,
                                                     const int32_t* __restrict__ slots,
                                                     const int32_t* __restrict__ positions,
                                                     PageGeom g, int32_t* status) {
  // block (b, i): token i of the gridDim.y new tokens of sequence b, written at position positions[b] + i
  const int b = blockIdx.x, i_tok = blockIdx.y, n_tok = gridDim.y;
  const int slot = slots ? slots[b] : b;
  const int pos = positions[b] + i_tok;
  if (slot < 0 || slot >= g.max_batch || positions[b] < 0 || pos >= g.max_pages_per_seq * g.page_tokens) {
    if (threadIdx.x == 0) report(status, ECHOKV_EBADPAGE);
    return;
  }
  const int page = g.table[(size_t)slot * g.max_pages_per_seq + pos / g.page_tokens];
  if (page < 0 || page >= g.n_pages) {
    if (threadIdx.x == 0) report(status, ECHOKV_EBADPAGE);
    return;
  }
  const size_t row = (size_t)page * g.page_tokens + pos % g.page_tokens;
  constexpr int kVec = 16 / sizeof(T);
  const uint4* ks = reinterpret_cast<const uint4*>(k_new + ((size_t)b * n_tok + i_tok) * D);
  const uint4* vs = reinterpret_cast<const uint4*>(v_new + ((size_t)b * n_tok + i_tok) * D);
  uint4* kd = reinterpret_cast<uint4*>(k_pool + row * (size_t)k_width);
  uint4* vd = reinterpret_cast<uint4*>(v_pool + row * (size_t)v_width);
  for (int i = threadIdx.x; i < k_width / kVec; i += blockDim.x) kd[i] = ks[i];
  for (int i = threadIdx.x; i < v_width / kVec; i += blockDim.x) vd[i] = vs[i];
}

cudaError_t launch_append(int dtype, void* k_pool, void* v_pool, int k_width, int v_width, int D, const void* k_new,
                          const void* v_new, const int32_t* slots, const int32_t* positions, int B, int n_tokens,
                          const PageGeom& geom, int32_t* status, cudaStream_t stream) {
  const dim3 grid(B, n_tokens);
  if (dtype == ECHOKV_BF16) {
    append_kernel<__nv_bfloat16><<<grid, 128, 0, stream>>>(
        (__nv_bfloat16*)k_pool, (__nv_bfloat16*)v_pool, k_width, v_width, D, (const __nv_bfloat16*)k_new,
        (const __nv_bfloat16*)v_new, slots, positions, geom, status);
  } else {
    append_kernel<float><<<grid, 128, 0, stream>>>((float*)k_pool, (float*)v_pool, k_width, v_width, D,
                                                (const float*)k_new, (const float*)v_new, slots,
                                                positions, geom, status);
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// The switch from full-cache generation to compressed inference (Section 3.1: compression is evicting
// part of each token's K / V; Section 5.4: done only once memory runs short, or during prefill): rows of a
// full-width cache are cut down to what a compressed layer keeps.  One block per (page of a sequence):
// dims 0 .. m-1 of every token go to the layer's pools (Eq. 2; the keys' first mk dims, mk = D where a layer keeps
// its keys whole), dims m .. D-1 of sink / window tokens to the side buffers (values only where the keys are
// whole).  Plain 16-byte copies: bit-exact.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) compress_kernel(const uint4* __restrict__ k_full, const uint4* __restrict__ v_full,
                                                       uint4* __restrict__ k_local, uint4* __restrict__ v_local,
                                                       uint4* __restrict__ k_side, uint4* __restrict__ v_side,
                                                       int d_vec, int mk_vec, int m_vec, int n_sink, int n_window,
                                                       const int32_t* __restrict__ slots,
                                                       const int32_t* __restrict__ begins,
                                                       const int32_t* __restrict__ lens, PageGeom g, int32_t* status) {
  const int b = blockIdx.y, page_idx = blockIdx.x, P = g.page_tokens;
  const int slot = slots ? slots[b] : b;
  const int len = lens[b];
  const int begin = begins ? begins[b] : 0;
  if (slot < 0 || slot >= g.max_batch) {
    if (threadIdx.x == 0 && page_idx == 0) report(status, ECHOKV_EBADPAGE);
    return;
  }
  if (len < 1 || len > g.max_pages_per_seq * P || begin < 0 || begin > len) {
    if (threadIdx.x == 0 && page_idx == 0) report(status, ECHOKV_EBADLENGTH);
    return;
  }
  const int t0 = page_idx * P;
  const int r_lo = max(begin - t0, 0), r_hi = min(len - t0, P);     // rows of this page to evict
  if (r_lo >= r_hi) return;
  const int page = g.table[(size_t)slot * g.max_pages_per_seq + page_idx];
  if (page < 0 || page >= g.n_pages) {
    if (threadIdx.x == 0) report(status, ECHOKV_EBADPAGE);
    return;
  }
  const size_t row0 = (size_t)page * P;
  if (mk_vec > 0) {
    for (int idx = r_lo * mk_vec + threadIdx.x; idx < r_hi * mk_vec; idx += blockDim.x) {
      const int r = idx / mk_vec, v = idx - r * mk_vec;
      k_local[(row0 + r) * mk_vec + v] = k_full[(row0 + r) * d_vec + v];
    }
  }
  if (m_vec > 0) {
    for (int idx = r_lo * m_vec + threadIdx.x; idx < r_hi * m_vec; idx += blockDim.x) {
      const int r = idx / m_vec, v = idx - r * m_vec;
      v_local[(row0 + r) * m_vec + v] = v_full[(row0 + r) * d_vec + v];
    }
  }
  const int drop_vec = d_vec - m_vec;
  if (v_side != nullptr && drop_vec > 0 && (t0 + r_lo < n_sink || t0 + r_hi > len - n_window)) {
    const size_t seq_base = (size_t)slot * (n_sink + n_window);
    for (int idx = r_lo * drop_vec + threadIdx.x; idx < r_hi * drop_vec; idx += blockDim.x) {
      const int r = idx / drop_vec, v = idx - r * drop_vec;
      const int t = t0 + r;
      const uint4 kv = k_full[(row0 + r) * d_vec + m_vec + v];
      const uint4 vv = v_full[(row0 + r) * d_vec + m_vec + v];
      if (t < n_sink) {
        if (k_side != nullptr) k_side[(seq_base + t) * drop_vec + v] = kv;
        v_side[(seq_base + t) * drop_vec + v] = vv;
      }
      if (n_window > 0 && t >= len - n_window) {
        if (k_side != nullptr) k_side[(seq_base + n_sink + t % n_window) * drop_vec + v] = kv;
        v_side[(seq_base + n_sink + t % n_window) * drop_vec + v] = vv;
      }
    }
  }
}

cudaError_t launch_compress(int elem_bytes, const void* k_full, const void* v_full, void* k_local, void* v_local,
                            const SideArgs* side, int D, int mk, int m, const int32_t* slots, const int32_t* begins,
                            const int32_t* lens, int B, const PageGeom& geom, int32_t* status, cudaStream_t stream) {
  const int d_vec = D * elem_bytes / 16, mk_vec = mk * elem_bytes / 16, m_vec = m * elem_bytes / 16;
  dim3 grid(geom.max_pages_per_seq, B);
  compress_kernel<<<grid, 256, 0, stream>>>(
      (const uint4*)k_full, (const uint4*)v_full, (uint4*)k_local, (uint4*)v_local,
      side ? (uint4*)side->k_side : nullptr, side ? (uint4*)side->v_side : nullptr, d_vec, mk_vec, m_vec,
      side ? side->n_sink : 0, side ? side->n_window : 0, slots, begins, lens, geom, status);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Attention over stored heads (Eq. 7 on the cache as stored): one warp per token row.
// ---------------------------------------------------------------------------------------------
template <typename T, int EPL>
__device__ __forceinline__ void load_row_slice(const T* p, float (&out)[EPL]) {
  if constexpr (sizeof(T) * EPL == 16) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    if constexpr (sizeof(T) == 4) {
      out[0] = __uint_as_float(v.x); out[1] = __uint_as_float(v.y);
      out[2] = __uint_as_float(v.z); out[3] = __uint_as_float(v.w);
    }
  } else if constexpr (sizeof(T) * EPL == 8) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    if constexpr (sizeof(T) == 4) {
      out[0] = __uint_as_float(v.x); out[1] = __uint_as_float(v.y);
    } else {
      out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xffff0000u);
      out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xffff0000u);
    }
  } else {
    static_assert(sizeof(T) * EPL == 4, "row slice of 4, 8 or 16 bytes");
    uint32_t v = *reinterpret_cast<const uint32_t*>(p);
    out[0] = __uint_as_float(v << 16); out[1] = __uint_as_float(v & 0xffff0000u);
  }
}

template <typename T, int DH, int G>
__global__ void __launch_bounds__(128) attn_stored_kernel(AttnArgs a, const T* __restrict__ k_pool,
                                                          const T* __restrict__ v_pool, int width,
                                                          int n_splits) {
  constexpr int EPL = DH / 32;
  constexpr int U = 4;   // tokens in flight per warp
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float sm_m[4][G], sm_l[4][G];
  __shared__ float sm_o[4][G][DH];

  int slot, len;
  {
    int32_t* st = threadIdx.x == 0 ? a.status : nullptr;
    slot = a.slots ? a.slots[b] : b;
    len = a.lens[b];
    const bool bad_slot = slot < 0 || slot >= a.geom.max_batch;
    const bool bad_len = len < 1 || len > a.geom.max_pages_per_seq * a.geom.page_tokens;
    if (bad_slot || bad_len) {
      if (st) report(st, bad_slot ? ECHOKV_EBADPAGE : ECHOKV_EBADLENGTH);
      return;
    }
  }
  const int P = a.geom.page_tokens;
  const int n_pages_seq = (len + P - 1) / P;
  const int pages_per_split = (n_pages_seq + n_splits - 1) / n_splits;
  const int t0 = split * pages_per_split * P;
  const int t1 = min(len, (split + 1) * pages_per_split * P);
  const int32_t* table = a.geom.table + (size_t)slot * a.geom.max_pages_per_seq;

  float qr[G][EPL];
  const T* q = reinterpret_cast<const T*>(a.q);
#pragma unroll
  for (int gi = 0; gi < G; ++gi) {
    float tmp[EPL];
    load_row_slice<T, EPL>(q + ((size_t)b * a.n_q_heads + kvh * G + gi) * DH + lane * EPL, tmp);
#pragma unroll
    for (int e = 0; e < EPL; ++e) qr[gi][e] = tmp[e] * a.scale_log2e;
  }
  // rotate-on-read: q . (R_t k) = sum_j k_j (q_j cos + sgn_j q_partner(j) sin), partner = j +- DH/2, which
  // lives 16 lanes away; sgn = +1 in the lower half of the head, -1 in the upper half
  const bool rope = a.rope.cs != nullptr;
  float qp[G][EPL];
#pragma unroll
  for (int gi = 0; gi < G; ++gi)
#pragma unroll
    for (int e = 0; e < EPL; ++e)
      qp[gi][e] = (lane < 16 ? 1.f : -1.f) * __shfl_xor_sync(0xffffffffu, qr[gi][e], 16);
  float m[G], l[G], o[G][EPL];
#pragma unroll
  for (int gi = 0; gi < G; ++gi) {
    m[gi] = -INFINITY;
    l[gi] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[gi][e] = 0.f;
  }

  for (int tb = t0 + warp * U; tb < t1; tb += 4 * U) {
    float kx[U][EPL], vx[U][EPL];
    bool valid[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int t = tb + u;
      valid[u] = t < t1;
      if (valid[u]) {
        const int page = table[t / P];
        if (page < 0 || page >= a.geom.n_pages) {
          if (lane == 0) report(a.status, ECHOKV_EBADPAGE);
          valid[u] = false;
        } else {
          const size_t off = ((size_t)page * P + t % P) * (size_t)width + kvh * DH + lane * EPL;
          load_row_slice<T, EPL>(k_pool + off, kx[u]);
          load_row_slice<T, EPL>(v_pool + off, vx[u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (!valid[u]) continue;   // warp-uniform
      float2 cs[EPL];
      if (rope) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) cs[e] = a.rope.cs[(size_t)((lane & 15) * EPL + e) * a.rope.stride + tb + u];
      }
#pragma unroll
      for (int gi = 0; gi < G; ++gi) {
        float s = 0.f;
        if (rope) {
#pragma unroll
          for (int e = 0; e < EPL; ++e) s = fmaf(kx[u][e], fmaf(qr[gi][e], cs[e].x, qp[gi][e] * cs[e].y), s);
        } else {
#pragma unroll
          for (int e = 0; e < EPL; ++e) s = fmaf(qr[gi][e], kx[u][e], s);
        }
        s = warp_sum(s);
        const float m_new = fmaxf(m[gi], s);
        const float alpha = exp2f(m[gi] - m_new);
        const float p = exp2f(s - m_new);
        l[gi] = l[gi] * alpha + p;
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[gi][e] = fmaf(p, vx[u][e], o[gi][e] * alpha);
        m[gi] = m_new;
      }
    }
  }

#pragma unroll
  for (int gi = 0; gi < G; ++gi) {
    if (lane == 0) {
      sm_m[warp][gi] = m[gi];
      sm_l[warp][gi] = l[gi];
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) sm_o[warp][gi][lane * EPL + e] = o[gi][e];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < G * DH; idx += 128) {
    const int gi = idx / DH, j = idx % DH;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) M = fmaxf(M, sm_m[w][gi]);
    float L = 0.f, acc = 0.f;
    if (M > -INFINITY) {
#pragma unroll
      for (int w = 0; w < 4; ++w) {
        const float wgt = exp2f(sm_m[w][gi] - M);
        L += wgt * sm_l[w][gi];
        acc += wgt * sm_o[w][gi][j];
      }
    }
    const size_t pidx = ((size_t)b * a.n_q_heads + kvh * G + gi) * a.parts.max_parts + split;
    a.parts.o[pidx * DH + j] = acc;
    if (j == 0) a.parts.ml[pidx] = make_float2(M, L);
  }
}

template <typename T, int DH>
static cudaError_t launch_attn_stored_g(const AttnArgs& a, const void* k_pool, const void* v_pool,
                                        int width, int n_heads, int n_splits, cudaStream_t stream) {
  const int g = a.n_q_heads / a.n_kv_heads;
  dim3 grid(n_splits, n_heads, a.batch);
  const T* kp = (const T*)k_pool;
  const T* vp = (const T*)v_pool;
  switch (g) {
    case 1: attn_stored_kernel<T, DH, 1><<<grid, 128, 0, stream>>>(a, kp, vp, width, n_splits); break;
    case 2: attn_stored_kernel<T, DH, 2><<<grid, 128, 0, stream>>>(a, kp, vp, width, n_splits); break;
    case 4: attn_stored_kernel<T, DH, 4><<<grid, 128, 0, stream>>>(a, kp, vp, width, n_splits); break;
    case 8: attn_stored_kernel<T, DH, 8><<<grid, 128, 0, stream>>>(a, kp, vp, width, n_splits); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_attn_stored(const AttnArgs& a, const void* k_pool, const void* v_pool, int width,
                               int n_heads, int n_splits, cudaStream_t stream) {
  if (n_heads == 0) return cudaSuccess;
  if (a.dtype == ECHOKV_BF16) {
    if (a.head_dim == 128)
      return launch_attn_stored_g<__nv_bfloat16, 128>(a, k_pool, v_pool, width, n_heads, n_splits, stream);
    return launch_attn_stored_g<__nv_bfloat16, 64>(a, k_pool, v_pool, width, n_heads, n_splits, stream);
  }
  if (a.head_dim == 128)
    return launch_attn_stored_g<float, 128>(a, k_pool, v_pool, width, n_heads, n_splits, stream);
  return launch_attn_stored_g<float, 64>(a, k_pool, v_pool, width, n_heads, n_splits, stream);
}

// ---------------------------------------------------------------------------------------------
// CUDA-core reconstruct-then-attend (Eq. 3, 6, 7 for one dropped KV head and one token range)
// ---------------------------------------------------------------------------------------------
constexpr int kKc = 32;   // features per staged chunk of the predictor input

template <int DH>
struct ReconSmem {
  float Xs[kKc][kSimtTileTokens];          // predictor-input chunk, [feature][token]
  float Ws[kKc][DH];                       // predictor chunk, [feature][output dim of the head]
  float Hs[kSimtTileTokens][DH + 1];       // predicted K (then V) tile of the head
  float Ss[kMaxGroup][kSimtTileTokens];    // scores, then probabilities
  float qs[kMaxGroup][DH];                 // queries * scale * log2e
  float kb[DH];                            // bias of the K predictor for this head (only with a rotation)
  float m_run[kMaxGroup], l_run[kMaxGroup], alpha[kMaxGroup];
};

// acc[8 tokens][FPT feats] += X[tile tokens][D_in] * W_head[DH][D_in]^T for one 64-token tile
template <typename T, int DH>
__device__ __forceinline__ void predict_tile(ReconSmem<DH>& sm, const T* __restrict__ anchor_pool,
                                             const T* __restrict__ local_pool,
                                             const T* __restrict__ W_head, int D, int m,
                                             const int32_t* __restrict__ table, const PageGeom& g,
                                             int tile_t0, int len, int32_t* status) {
  constexpr int FPT = DH / 16;
  constexpr int KPT = kKc * DH / 128;          // predictor k-values loaded per thread and chunk
  constexpr int VN = Vec16<T>::N;
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  float acc[8][FPT];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < FPT; ++j) acc[i][j] = 0.f;

  // this thread stages 16 features of token (tid / 2)
  const int ld_tok = tid / 2, ld_half = tid % 2;
  const int t_glob = tile_t0 + ld_tok;
  long long row = -1;   // row index inside a pool, or -1 for a padding token
  if (t_glob < len) {
    const int page = table[t_glob / g.page_tokens];
    if (page < 0 || page >= g.n_pages) {
      report(status, ECHOKV_EBADPAGE);
    } else {
      row = (long long)page * g.page_tokens + t_glob % g.page_tokens;
    }
  }
  const int w_row = tid % DH, w_part = tid / DH;
  const int d_in = D + m;

  for (int kc = 0; kc < d_in; kc += kKc) {
    // stage X chunk (transposed) and W chunk (transposed)
    {
      float xv[16];
      if (row >= 0) {
        const T* src = kc < D ? anchor_pool + row * D + kc : local_pool + row * m + (kc - D);
        src += ld_half * 16;
#pragma unroll
        for (int v = 0; v < 16 / VN; ++v) Vec16<T>::load(src + v * VN, xv + v * VN);
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) xv[e] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < 16; ++e) sm.Xs[ld_half * 16 + e][ld_tok] = xv[e];
      float wv[KPT];
      const T* wsrc = W_head + (size_t)w_row * d_in + kc + w_part * KPT;
#pragma unroll
      for (int v = 0; v < KPT / VN; ++v) Vec16<T>::load(wsrc + v * VN, wv + v * VN);
#pragma unroll
      for (int e = 0; e < KPT; ++e) sm.Ws[w_part * KPT + e][w_row] = wv[e];
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < kKc; ++k) {
      float xr[8], wr[FPT];
#pragma unroll
      for (int i = 0; i < 8; ++i) xr[i] = sm.Xs[k][ty * 8 + i];
#pragma unroll
      for (int j = 0; j < FPT; ++j) wr[j] = sm.Ws[k][tx * FPT + j];
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < FPT; ++j) acc[i][j] = fmaf(xr[i], wr[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < FPT; ++j) sm.Hs[ty * 8 + i][tx * FPT + j] = acc[i][j];
}

template <typename T, int DH>
__global__ void __launch_bounds__(128) recon_simt_kernel(AttnArgs a, ReconArgs r) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  ReconSmem<DH>& sm = *reinterpret_cast<ReconSmem<DH>*>(smem_raw);
  const int part = blockIdx.x, b = blockIdx.z;
  const int n_ret = retained_heads(r, DH);
  const int kvh = n_ret + blockIdx.y;                 // dropped KV head
  const int g = a.n_q_heads / a.n_kv_heads;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  const int slot = a.slots ? a.slots[b] : b;
  const int len = a.lens[b];
  if (slot < 0 || slot >= a.geom.max_batch) {
    if (tid == 0) report(a.status, ECHOKV_EBADPAGE);
    return;
  }
  if (len < 1 || len > r.capacity_tokens) {
    if (tid == 0) report(a.status, ECHOKV_EBADLENGTH);
    return;
  }
  const int part_t0 = part * r.part_tokens;
  if (part_t0 >= len) return;
  const int32_t* table = a.geom.table + (size_t)slot * a.geom.max_pages_per_seq;

  const T* q = reinterpret_cast<const T*>(a.q);
  for (int idx = tid; idx < g * DH; idx += 128) {
    const int gi = idx / DH, j = idx % DH;
    sm.qs[gi][j] = to_f32(q[((size_t)b * a.n_q_heads + kvh * g + gi) * DH + j]) * a.scale_log2e;
  }
  if (tid < kMaxGroup) {
    sm.m_run[tid] = -INFINITY;
    sm.l_run[tid] = 0.f;
  }
  // (a bias on predicted keys is rotated with them, so it does not cancel in the softmax then)
  for (int j = tid; j < DH; j += 128)
    sm.kb[j] = r.bk != nullptr ? to_f32(reinterpret_cast<const T*>(r.bk)[(size_t)(kvh - n_ret) * DH + j]) : 0.f;
  float o[kMaxGroup];
#pragma unroll
  for (int gi = 0; gi < kMaxGroup; ++gi) o[gi] = 0.f;
  __syncthreads();

  const size_t w_off = (size_t)(kvh - n_ret) * DH * (r.D + r.m);
  const T* Wk_head = reinterpret_cast<const T*>(r.Wk) + w_off;
  const T* Wv_head = reinterpret_cast<const T*>(r.Wv) + w_off;
  const int tiles = r.part_tokens / kSimtTileTokens;

  for (int tile = 0; tile < tiles; ++tile) {
    const int tile_t0 = part_t0 + tile * kSimtTileTokens;
    if (tile_t0 >= len) break;
    // K_hat tile (Eq. 3) -> Hs
    predict_tile<T, DH>(sm, (const T*)r.k_anchor, (const T*)r.k_local, Wk_head, r.D, r.m, table,
                        a.geom, tile_t0, len, a.status);
    __syncthreads();
    // scores of the group's query heads (Eq. 7), base-2 units
    {
      const int t = tid % kSimtTileTokens;
      for (int gi = tid / kSimtTileTokens; gi < g; gi += 128 / kSimtTileTokens) {
        const int t_seq = tile_t0 + t;     // predicted tokens only (sink / window tokens come from the side buffers)
        float s = 0.f;
        if (a.rope.cs != nullptr) {
          // the predicted key row is rotated to position t_seq before q . k
          const float2* cs = a.rope.cs + min(t_seq, a.rope.stride - 1);
#pragma unroll 8
          for (int j = 0; j < DH / 2; ++j) {
            const float2 w = cs[(size_t)j * a.rope.stride];
            const float k_lo = sm.Hs[t][j] + sm.kb[j], k_hi = sm.Hs[t][j + DH / 2] + sm.kb[j + DH / 2];
            s = fmaf(sm.qs[gi][j], k_lo * w.x - k_hi * w.y, s);
            s = fmaf(sm.qs[gi][j + DH / 2], k_hi * w.x + k_lo * w.y, s);
          }
        } else {
#pragma unroll 8
          for (int j = 0; j < DH; ++j) s = fmaf(sm.qs[gi][j], sm.Hs[t][j], s);
        }
        sm.Ss[gi][t] = (t_seq >= predicted_lo(len, r.n_sink) && t_seq < predicted_hi(len, r.n_sink, r.n_window))
                           ? s : -INFINITY;
      }
    }
    __syncthreads();
    // online softmax update, one warp per query head
    for (int gi = warp; gi < g; gi += 4) {
      const float s0 = sm.Ss[gi][lane], s1 = sm.Ss[gi][lane + 32];
      const float mt = warp_max(fmaxf(s0, s1));
      const float m_old = sm.m_run[gi];
      const float m_new = fmaxf(m_old, mt);
      const float m_use = m_new == -INFINITY ? 0.f : m_new;     // nothing predicted so far: every p is 0
      const float alpha = exp2f(m_old - m_use);
      const float p0 = exp2f(s0 - m_use), p1 = exp2f(s1 - m_use);
      const float ls = warp_sum(p0 + p1);
      sm.Ss[gi][lane] = p0;
      sm.Ss[gi][lane + 32] = p1;
      if (lane == 0) {
        sm.m_run[gi] = m_new;
        sm.l_run[gi] = sm.l_run[gi] * alpha + ls;
        sm.alpha[gi] = alpha;
      }
    }
    __syncthreads();   // Hs (K_hat) fully consumed, Ss holds probabilities
    // V_hat tile (Eq. 3) -> Hs
    predict_tile<T, DH>(sm, (const T*)r.v_anchor, (const T*)r.v_local, Wv_head, r.D, r.m, table,
                        a.geom, tile_t0, len, a.status);
    __syncthreads();
    if (tid < DH) {
      for (int gi = 0; gi < g; ++gi) {
        float acc = o[gi] * sm.alpha[gi];
#pragma unroll 8
        for (int t = 0; t < kSimtTileTokens; ++t) acc = fmaf(sm.Ss[gi][t], sm.Hs[t][tid], acc);
        o[gi] = acc;
      }
    }
    __syncthreads();
  }

  for (int gi = 0; gi < g; ++gi) {
    const size_t pidx = ((size_t)b * a.n_q_heads + kvh * g + gi) * a.parts.max_parts + part;
    if (tid < DH) a.parts.o[pidx * DH + tid] = o[gi];
    if (tid == 0) a.parts.ml[pidx] = make_float2(sm.m_run[gi], sm.l_run[gi]);
  }
}

template <typename T, int DH>
static cudaError_t launch_recon_simt_t(const AttnArgs& a, const ReconArgs& r, cudaStream_t stream) {
  const int n_drop = a.n_kv_heads - retained_heads(r, DH);
  const int n_parts = (r.capacity_tokens + r.part_tokens - 1) / r.part_tokens;
  const size_t smem = sizeof(ReconSmem<DH>);
  cudaError_t e = cudaFuncSetAttribute(recon_simt_kernel<T, DH>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(n_parts, n_drop, a.batch);
  recon_simt_kernel<T, DH><<<grid, 128, smem, stream>>>(a, r);
  return cudaGetLastError();
}

cudaError_t launch_recon_simt(const AttnArgs& a, const ReconArgs& r, cudaStream_t stream) {
  if (a.n_q_heads / a.n_kv_heads > kMaxGroup) return cudaErrorInvalidValue;
  if (a.dtype == ECHOKV_BF16) {
    if (a.head_dim == 128) return launch_recon_simt_t<__nv_bfloat16, 128>(a, r, stream);
    return launch_recon_simt_t<__nv_bfloat16, 64>(a, r, stream);
  }
  if (a.head_dim == 128) return launch_recon_simt_t<float, 128>(a, r, stream);
  return launch_recon_simt_t<float, 64>(a, r, stream);
}

// ---------------------------------------------------------------------------------------------
// Split-K merge: log-sum-exp combination of partial (max, sum, weighted V) triples
// ---------------------------------------------------------------------------------------------
constexpr int kMergeGroups = 4;   // partials are dealt round-robin to this many thread groups

template <typename T>
__global__ void __launch_bounds__(128 * kMergeGroups)
merge_kernel(AttnArgs a, float* __restrict__ out, int n_stored_heads, int n_stored_parts,
             const int32_t* __restrict__ stored_item_tokens, int stored_batch_per_slot, int part_tokens,
             const T* __restrict__ bv, const T* __restrict__ bk_shift, int extra_recon_part,
             const int32_t* __restrict__ choose, int alt_part_tokens) {
  if (choose != nullptr && *choose == 1) part_tokens = alt_part_tokens;
  const int h = blockIdx.x, b = blockIdx.y, j = threadIdx.x, grp = threadIdx.y;
  const int DH = a.head_dim;                      // == blockDim.x
  const int tid = grp * DH + j, n_threads = DH * kMergeGroups;
  const size_t oidx = ((size_t)b * a.n_q_heads + h) * DH + j;
  const int slot = a.slots ? a.slots[b] : b;
  const int len = a.lens[b];
  if (slot < 0 || slot >= a.geom.max_batch || len < 1 ||
      len > a.geom.max_pages_per_seq * a.geom.page_tokens) {      // (the same for the whole block)
    if (grp == 0) out[oidx] = 0.f;
    return;
  }
  const int g = a.n_q_heads / a.n_kv_heads;
  const int kvh = h / g;
  const bool stored = kvh < n_stored_heads;
  int n;
  if (!stored) {
    n = (len + part_tokens - 1) / part_tokens + extra_recon_part;   // (+ the sink / window partial)
  } else if (stored_item_tokens != nullptr) {
    const int item_tokens = stored_item_tokens[b / stored_batch_per_slot];
    n = (len + item_tokens - 1) / item_tokens;
  } else {
    n = n_stored_parts;
  }
  const size_t base = ((size_t)b * a.n_q_heads + h) * a.parts.max_parts;
  __shared__ float s_max[16];
  __shared__ float s_l[kMergeGroups];
  __shared__ float s_l_side[kMergeGroups];
  __shared__ float s_acc[kMergeGroups][128];
  // (the sink / window partial of a predicted head is its last one: those tokens' keys and values are the true ones)
  const int side_part = (!stored && extra_recon_part) ? n - 1 : -1;
  // A bias on the K predictor shifts the scores of a head's predicted tokens by q . b_k: it cancels in the softmax
  // unless sink / window tokens, whose keys are not predicted, take part; then the predicted partials move by it.
  // (bk_shift is null when nothing has to move, and when the kernels added the bias themselves: rotated keys.)
  float shift = 0.f;
  if (bk_shift != nullptr && side_part >= 0) {
    __shared__ float s_dot[4];
    const T* qrow = reinterpret_cast<const T*>(a.q) + ((size_t)b * a.n_q_heads + h) * DH;
    float d = grp == 0 ? to_f32(qrow[j]) * to_f32(bk_shift[(kvh - n_stored_heads) * DH + j]) : 0.f;
    d = warp_sum(d);
    if (grp == 0 && (j & 31) == 0) s_dot[j >> 5] = d;
    __syncthreads();
    for (int w = 0; w < DH / 32; ++w) shift += s_dot[w];
    shift *= a.scale_log2e;
  }
  // pass 1: the largest partial maximum, all threads of the block together
  float m = -INFINITY;
  for (int p = tid; p < n; p += n_threads) m = fmaxf(m, a.parts.ml[base + p].x + (p == side_part ? 0.f : shift));
  m = warp_max(m);
  if ((tid & 31) == 0) s_max[tid >> 5] = m;
  __syncthreads();
  float M = -INFINITY;
  for (int w = 0; w < n_threads / 32; ++w) M = fmaxf(M, s_max[w]);
  // pass 2: each group sums every kMergeGroups-th partial
  float L = 0.f, L_side = 0.f, acc = 0.f;
  if (M > -INFINITY) {
#pragma unroll 4
    for (int p = grp; p < n; p += kMergeGroups) {
      const float2 ml = a.parts.ml[base + p];
      const float w = exp2f(ml.x + (p == side_part ? 0.f : shift) - M);
      L = fmaf(w, ml.y, L);
      if (p == side_part) L_side = w * ml.y;
      acc = fmaf(w, a.parts.o[(base + p) * DH + j], acc);
    }
  }
  s_acc[grp][j] = acc;
  if (j == 0) {
    s_l[grp] = L;
    s_l_side[grp] = L_side;
  }
  __syncthreads();
  if (grp != 0) return;
#pragma unroll
  for (int k = 1; k < kMergeGroups; ++k) {
    acc += s_acc[k][j];
    L += s_l[k];
    L_side += s_l_side[k];
  }
  float res = L > 0.f ? acc / L : 0.f;
  // A bias on the V predictor shifts every predicted V row alike, so it adds to the output weighted by the
  // probability of the predicted tokens: all of it (sum_t p_t = 1) unless sink / window tokens, whose values are not
  // predicted, take their share.  A bias on the K predictor shifts all scores of a head by the same amount and
  // cancels in the softmax (without a rotation).
  if (bv != nullptr && !stored && L > 0.f) res += to_f32(bv[(kvh - n_stored_heads) * DH + j]) * ((L - L_side) / L);
  out[oidx] = res;
}

cudaError_t launch_merge(const AttnArgs& a, float* out, int n_stored_heads, int n_stored_parts,
                         const int32_t* stored_item_tokens, int stored_batch_per_slot, int part_tokens,
                         const void* bv, cudaStream_t stream, int extra_recon_part, const void* bk_shift,
                         const int32_t* choose, int alt_part_tokens) {
  dim3 grid(a.n_q_heads, a.batch);
  if (a.dtype == ECHOKV_BF16) {
    merge_kernel<__nv_bfloat16><<<grid, dim3(a.head_dim, kMergeGroups), 0, stream>>>(
        a, out, n_stored_heads, n_stored_parts, stored_item_tokens, stored_batch_per_slot, part_tokens,
        (const __nv_bfloat16*)bv, (const __nv_bfloat16*)bk_shift, extra_recon_part, choose, alt_part_tokens);
  } else {
    merge_kernel<float><<<grid, dim3(a.head_dim, kMergeGroups), 0, stream>>>(a, out, n_stored_heads, n_stored_parts,
                                                         stored_item_tokens, stored_batch_per_slot,
                                                         part_tokens, (const float*)bv, (const float*)bk_shift,
                                                         extra_recon_part, choose, alt_part_tokens);
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// A retained width m that splits a head (Eq. 6 concatenates at the flat index m, wherever it falls): the
// explicit kernels work on whole heads, so the split head is treated as predicted and its stored dims are
// passed through the predictor by `split` one-hot rows put in front of W -- row i < split copies local dim
// m_heads + i (input column D + m_heads + i); multiplying a stored bf16 / fp32 value by 1 and adding zeros
// is exact, so the rebuilt head holds the stored dims bit for bit.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) extend_predictor_kernel(const T* __restrict__ W, const T* __restrict__ bias,
                                                               T* __restrict__ Wx, T* __restrict__ bx, int d_in,
                                                               int split, int pass_col0) {
  const int row = blockIdx.x;                       // row of the extended matrix
  T* dst = Wx + (size_t)row * d_in;
  if (row < split) {
    for (int c = threadIdx.x; c < d_in; c += blockDim.x) dst[c] = c == pass_col0 + row ? T(1.0f) : T(0.0f);
  } else {
    const T* src = W + (size_t)(row - split) * d_in;
    for (int c = threadIdx.x; c < d_in; c += blockDim.x) dst[c] = src[c];
  }
  if (threadIdx.x == 0 && bx != nullptr) bx[row] = (row < split || bias == nullptr) ? T(0.0f) : bias[row - split];
}

cudaError_t launch_extend_predictor(int dtype, const void* W, const void* bias, void* Wx, void* bx, int d_drop,
                                    int d_in, int split, int pass_col0, cudaStream_t stream) {
  const int rows = d_drop + split;
  if (dtype == ECHOKV_BF16)
    extend_predictor_kernel<__nv_bfloat16><<<rows, 256, 0, stream>>>((const __nv_bfloat16*)W, (const __nv_bfloat16*)bias,
                                                                  (__nv_bfloat16*)Wx, (__nv_bfloat16*)bx, d_in, split,
                                                                  pass_col0);
  else
    extend_predictor_kernel<float><<<rows, 256, 0, stream>>>((const float*)W, (const float*)bias, (float*)Wx, (float*)bx,
                                                          d_in, split, pass_col0);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Sink and recent-window tokens at full precision (Section 4.1): their dropped dims live in small
// side buffers; these two kernels write and attend them.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) append_side_kernel(T* __restrict__ k_side, T* __restrict__ v_side, int n_sink,
                                                          int n_window, int d_drop, int m, int D,
                                                          const T* __restrict__ k_new, const T* __restrict__ v_new,
                                                          const int32_t* __restrict__ slots,
                                                          const int32_t* __restrict__ positions, int max_batch,
                                                          int32_t* status) {
  // block (b, i): token i of the gridDim.y new tokens of sequence b, at position positions[b] + i
  const int b = blockIdx.x, i_tok = blockIdx.y, n_tok = gridDim.y;
  const int slot = slots ? slots[b] : b;
  const int pos = positions[b] + i_tok;
  if (slot < 0 || slot >= max_batch || positions[b] < 0) {
    if (threadIdx.x == 0) report(status, ECHOKV_EBADPAGE);
    return;
  }
  constexpr int kVec = 16 / sizeof(T);
  const int n_vec = d_drop / kVec;
  const uint4* ks = reinterpret_cast<const uint4*>(k_new + ((size_t)b * n_tok + i_tok) * D + m);
  const uint4* vs = reinterpret_cast<const uint4*>(v_new + ((size_t)b * n_tok + i_tok) * D + m);
  const size_t seq_base = (size_t)slot * (n_sink + n_window);
  // a token inside the sink is written there; every token also enters the window ring -- of a chunk only the
  // last n_window tokens, which are the ones that remain in it (and no two of them share a ring slot)
  for (int which = 0; which < 2; ++which) {
    int idx;
    if (which == 0) { if (pos >= n_sink) continue; idx = pos; }
    else { if (n_window == 0 || i_tok < n_tok - n_window) continue; idx = n_sink + pos % n_window; }
    uint4* kd = k_side != nullptr ? reinterpret_cast<uint4*>(k_side + (seq_base + idx) * d_drop) : nullptr;
    uint4* vd = reinterpret_cast<uint4*>(v_side + (seq_base + idx) * d_drop);
    for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
      if (kd != nullptr) kd[i] = ks[i];        // (no K side buffer where the keys are kept whole)
      vd[i] = vs[i];
    }
  }
}

cudaError_t launch_append_side(int dtype, const SideArgs& side, int m, int D, const void* k_new, const void* v_new,
                               const int32_t* slots, const int32_t* positions, int B, int n_tokens, int max_batch,
                               int32_t* status, cudaStream_t stream) {
  const dim3 grid(B, n_tokens);
  if (dtype == ECHOKV_BF16) {
    append_side_kernel<__nv_bfloat16><<<grid, 128, 0, stream>>>(
        (__nv_bfloat16*)side.k_side, (__nv_bfloat16*)side.v_side, side.n_sink, side.n_window, side.d_drop, m, D,
        (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, slots, positions, max_batch, status);
  } else {
    append_side_kernel<float><<<grid, 128, 0, stream>>>((float*)side.k_side, (float*)side.v_side, side.n_sink,
                                                     side.n_window, side.d_drop, m, D, (const float*)k_new,
                                                     (const float*)v_new, slots, positions, max_batch, status);
  }
  return cudaGetLastError();
}

// One block per (KV head, sequence): scores of the <= n_sink + n_window full-precision tokens against the
// group's query heads, softmax, weighted V; one partial per query head.  Of a head's DH dims the first
// n_stored = clamp(m - head * DH, 0, DH) are read from the layer's pool (row width m) and the rest from the side
// buffers (dims m .. D-1): a dropped head reads the side buffers only, a head that m splits reads half and half, a
// retained head (only asked for by the absorbed mode, first_head = 0) reads the pool only.  The K pool may be wider
// than the V pool (mk > m: keys kept whole); the keys' side buffer is then not read at all.
// The partial goes to index fixed_part, or ceil(len / part_tokens) if that is < 0.
constexpr int kSideThreads = 160;      // the paper's 4 + 128 full-precision tokens in one pass of a token per thread
constexpr int kSideWarps = kSideThreads / 32;
// four consecutive stored elements, widened to fp32
__device__ __forceinline__ void load4(const float* p, float (&out)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
__device__ __forceinline__ void load4(const __nv_bfloat16* p, float (&out)[4]) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xffff0000u);
  out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xffff0000u);
}

template <typename T, int DH>
__global__ void __launch_bounds__(kSideThreads) attn_side_kernel(AttnArgs a, const T* __restrict__ k_side,
                                                        const T* __restrict__ v_side, int n_sink, int n_window,
                                                        int d_drop, int mk, int m, int part_tokens, int first_head,
                                                        int fixed_part, const T* __restrict__ k_pool,
                                                        const T* __restrict__ v_pool,
                                                        const int32_t* __restrict__ choose, int alt_part_tokens) {
  if (choose != nullptr && *choose == 1) part_tokens = alt_part_tokens;
  extern __shared__ float side_smem[];
  const int b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = a.n_q_heads / a.n_kv_heads;
  const int kvh = first_head + blockIdx.x;
  const int n_stored_k = min(max(mk - kvh * DH, 0), DH);  // 0, DH / 2 or DH (m is a multiple of 64)
  const int n_stored = min(max(m - kvh * DH, 0), DH);     // the same for the values
  const int n_side = n_sink + n_window;
  float* qs = side_smem;                      // [g][DH]
  float* sc = qs + kMaxGroup * DH;            // [g][n_side]
  // element offsets of every full-precision token's row: [0] in the K pool, [1] in the V pool (the head's dim 0),
  // [2] in the side buffers (dim m)
  unsigned long long* rows = reinterpret_cast<unsigned long long*>(sc + kMaxGroup * n_side);   // [3][n_side]
  float* osum = reinterpret_cast<float*>(rows + 3 * n_side);                                   // [g][DH]
  __shared__ float red[kSideWarps][kMaxGroup];
  __shared__ float s_m[kMaxGroup], s_l[kMaxGroup];
  const int slot = a.slots ? a.slots[b] : b;
  const int len = a.lens[b];
  if (slot < 0 || slot >= a.geom.max_batch || len < 1 ||
      len > a.geom.max_pages_per_seq * a.geom.page_tokens)
    return;                                    // (reported by the other kernels of the call; merge writes zeros)
  const int lo = predicted_lo(len, n_sink), hi = predicted_hi(len, n_sink, n_window);
  const int n_tok = lo + (len - hi);          // sink tokens [0, lo) then window tokens [hi, len)
  const T* q = reinterpret_cast<const T*>(a.q);
  for (int idx = tid; idx < g * DH; idx += kSideThreads)
    qs[idx] = to_f32(q[((size_t)b * a.n_q_heads + kvh * g) * DH + idx]) * a.scale_log2e;
  __syncthreads();
  const size_t seq_base = (size_t)slot * n_side;
  const int32_t* table = a.geom.table + (size_t)slot * a.geom.max_pages_per_seq;
  // where each full-precision token lives (looked up once: the loops below must not chase the block table)
  for (int i = tid; i < n_tok; i += kSideThreads) {
    const int t = i < lo ? i : hi + (i - lo);
    if (n_stored_k > 0) {
      int page = table[t / a.geom.page_tokens];
      if (page < 0 || page >= a.geom.n_pages) {
        report(a.status, ECHOKV_EBADPAGE);
        page = 0;
      }
      const size_t r = (size_t)page * a.geom.page_tokens + t % a.geom.page_tokens;
      rows[i] = r * (size_t)mk + (size_t)kvh * DH;
      rows[n_side + i] = r * (size_t)m + (size_t)kvh * DH;
    }
    // (offset of flat dim m; a head's first dim that is not stored is added where it is read)
    rows[2 * n_side + i] = (seq_base + (t < lo ? t : n_sink + t % n_window)) * (size_t)d_drop;
  }
  __syncthreads();
  // address of dims [j, j + vector) of token i's key / value row (a vector never straddles n_stored)
  auto k_at = [&](int i, int j) -> const T* {
    return j < n_stored_k ? k_pool + rows[i] + j : k_side + rows[2 * n_side + i] + (kvh * DH + j - mk);
  };
  // scores: one token per thread
  for (int i = tid; i < n_tok; i += kSideThreads) {
    float acc[kMaxGroup];
#pragma unroll
    for (int gi = 0; gi < kMaxGroup; ++gi) acc[gi] = 0.f;
    if (a.rope.cs != nullptr) {
      // the key row is rotated to its position before q . k
      const float2* cs = a.rope.cs + (i < lo ? i : hi + (i - lo));
      for (int j = 0; j < DH / 2; j += Vec16<T>::N) {
        float k_lo[Vec16<T>::N], k_hi[Vec16<T>::N];
        Vec16<T>::load(k_at(i, j), k_lo);
        Vec16<T>::load(k_at(i, DH / 2 + j), k_hi);
#pragma unroll
        for (int e = 0; e < Vec16<T>::N; ++e) {
          const float2 w = cs[(size_t)(j + e) * a.rope.stride];
          const float r_lo = k_lo[e] * w.x - k_hi[e] * w.y, r_hi = k_hi[e] * w.x + k_lo[e] * w.y;
#pragma unroll
          for (int gi = 0; gi < kMaxGroup; ++gi)
            if (gi < g) acc[gi] = fmaf(r_hi, qs[gi * DH + DH / 2 + j + e], fmaf(r_lo, qs[gi * DH + j + e], acc[gi]));
        }
      }
    } else {
      for (int j = 0; j < DH; j += Vec16<T>::N) {
        float kv[Vec16<T>::N];
        Vec16<T>::load(k_at(i, j), kv);
#pragma unroll
        for (int gi = 0; gi < kMaxGroup; ++gi)
          if (gi < g) {
#pragma unroll
            for (int e = 0; e < Vec16<T>::N; ++e) acc[gi] = fmaf(kv[e], qs[gi * DH + j + e], acc[gi]);
          }
      }
    }
#pragma unroll
    for (int gi = 0; gi < kMaxGroup; ++gi)
      if (gi < g) sc[gi * n_side + i] = acc[gi];
  }
  __syncthreads();
  // max and sum per query head
  for (int gi = 0; gi < g; ++gi) {
    float mx = -INFINITY;
    for (int i = tid; i < n_tok; i += kSideThreads) mx = fmaxf(mx, sc[gi * n_side + i]);
    mx = warp_max(mx);
    if (lane == 0) red[warp][gi] = mx;
  }
  __syncthreads();
  if (tid < g) {
    float mx = red[0][tid];
    for (int wi = 1; wi < kSideWarps; ++wi) mx = fmaxf(mx, red[wi][tid]);
    s_m[tid] = mx;
  }
  __syncthreads();
  for (int gi = 0; gi < g; ++gi) {
    const float M = s_m[gi];
    float l = 0.f;
    for (int i = tid; i < n_tok; i += kSideThreads) {
      const float pv = exp2f(sc[gi * n_side + i] - M);
      sc[gi * n_side + i] = pv;
      l += pv;
    }
    l = warp_sum(l);
    if (lane == 0) red[warp][gi] = l;
  }
  __syncthreads();
  if (tid < g) {
    float l = 0.f;
    for (int wi = 0; wi < kSideWarps; ++wi) l += red[wi][tid];
    s_l[tid] = l;
  }
  for (int idx = tid; idx < g * DH; idx += kSideThreads) osum[idx] = 0.f;
  __syncthreads();
  // weighted V: four output features per lane, warp s on the tokens s, s + 5, ..., four loads in flight; the
  // warps' sums are added up in shared memory, one warp after the other
  const int part = fixed_part >= 0 ? fixed_part : (len + part_tokens - 1) / part_tokens;
  {
    const int d0 = 4 * lane;                     // (a group of four dims never straddles n_stored: a multiple of 64)
    const bool active = d0 < DH;
    const bool from_pool = d0 < n_stored;
    const T* v_src = from_pool ? v_pool + d0 : v_side + (kvh * DH + d0 - m);
    const unsigned long long* v_rows = from_pool ? rows + n_side : rows + 2 * n_side;
    float o[kMaxGroup][4];
#pragma unroll
    for (int gi = 0; gi < kMaxGroup; ++gi)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[gi][e] = 0.f;
    for (int i0 = warp; active && i0 < n_tok; i0 += 4 * kSideWarps) {
      float vv[4][4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kSideWarps;
        if (i < n_tok) load4(v_src + v_rows[i], vv[u]);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * kSideWarps;
        if (i < n_tok) {
#pragma unroll
          for (int gi = 0; gi < kMaxGroup; ++gi)
            if (gi < g) {
              const float pv = sc[gi * n_side + i];
#pragma unroll
              for (int e = 0; e < 4; ++e) o[gi][e] = fmaf(pv, vv[u][e], o[gi][e]);
            }
        }
      }
    }
    for (int sl = 0; sl < kSideWarps; ++sl) {
      if (warp == sl && active) {
#pragma unroll
        for (int gi = 0; gi < kMaxGroup; ++gi)
          if (gi < g) {
#pragma unroll
            for (int e = 0; e < 4; ++e) osum[gi * DH + d0 + e] += o[gi][e];
          }
      }
      __syncthreads();
    }
  }
  for (int idx = tid; idx < g * DH; idx += kSideThreads) {
    const int gi = idx / DH, d = idx - gi * DH;
    const size_t pidx = ((size_t)b * a.n_q_heads + kvh * g + gi) * a.parts.max_parts + part;
    a.parts.o[pidx * DH + d] = osum[idx];
    if (d == 0) a.parts.ml[pidx] = make_float2(s_m[gi], s_l[gi]);
  }
}

template <typename T, int DH>
static cudaError_t launch_attn_side_t(const AttnArgs& a, const SideArgs& side, int first_head, int part_tokens,
                                      cudaStream_t stream, const SidePool& pool, const int32_t* choose,
                                      int alt_part_tokens) {
  const int n_heads = a.n_kv_heads - first_head;
  const int n_side = side.n_sink + side.n_window;
  const size_t smem = (size_t)(2 * kMaxGroup * DH + kMaxGroup * n_side) * sizeof(float) + (size_t)n_side * 24 + 8;
  cudaError_t e = cudaFuncSetAttribute(attn_side_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (n_heads <= 0) return cudaSuccess;
  dim3 grid(n_heads, a.batch);
  attn_side_kernel<T, DH><<<grid, kSideThreads, smem, stream>>>(
      a, (const T*)side.k_side, (const T*)side.v_side, side.n_sink, side.n_window, side.d_drop,
      pool.k_width > 0 ? pool.k_width : pool.width, pool.width, part_tokens, first_head, pool.part,
      (const T*)pool.k_pool, (const T*)pool.v_pool, choose, alt_part_tokens);
  return cudaGetLastError();
}

cudaError_t launch_attn_side(const AttnArgs& a, const SideArgs& side, int first_head, int part_tokens,
                             cudaStream_t stream, const SidePool& pool, const int32_t* choose, int alt_part_tokens) {
  if (a.dtype == ECHOKV_BF16) {
    if (a.head_dim == 128)
      return launch_attn_side_t<__nv_bfloat16, 128>(a, side, first_head, part_tokens, stream, pool, choose,
                                                    alt_part_tokens);
    return launch_attn_side_t<__nv_bfloat16, 64>(a, side, first_head, part_tokens, stream, pool, choose, alt_part_tokens);
  }
  if (a.head_dim == 128)
    return launch_attn_side_t<float, 128>(a, side, first_head, part_tokens, stream, pool, choose, alt_part_tokens);
  return launch_attn_side_t<float, 64>(a, side, first_head, part_tokens, stream, pool, choose, alt_part_tokens);
}

// ---------------------------------------------------------------------------------------------
// Are the pages of the batch's sequences consecutive in the pool?  (see launch_page_order)
// ---------------------------------------------------------------------------------------------
constexpr int kOrderSamplesPerSeq = 256;
__global__ void __launch_bounds__(256) page_order_kernel(const int32_t* __restrict__ slots,
                                                         const int32_t* __restrict__ lens, int batch, PageGeom g,
                                                         int32_t* __restrict__ flag) {
  __shared__ int s_in_order, s_seen;
  if (threadIdx.x == 0) s_in_order = s_seen = 0;
  __syncthreads();
  const int per_group = 64 / g.page_tokens;          // pages of an aligned 64-token group (page_tokens <= 32)
  int in_order = 0, seen = 0;
  for (int b = 0; b < batch; ++b) {
    const int slot = slots ? slots[b] : b;
    const int len = lens[b];
    if (slot < 0 || slot >= g.max_batch || len < 1 || len > g.max_pages_per_seq * g.page_tokens) continue;
    const int n_groups = len / 64;                    // whole groups only
    const int n_samples = min(n_groups, kOrderSamplesPerSeq);
    const int32_t* table = g.table + (size_t)slot * g.max_pages_per_seq;
    for (int i = threadIdx.x; i < n_samples; i += blockDim.x) {
      const int grp = (int)((long long)i * n_groups / n_samples);
      const int p0 = table[grp * per_group];
      bool ok = true;
      for (int k = 1; k < per_group; ++k) ok = ok && table[grp * per_group + k] == p0 + k;
      in_order += ok ? 1 : 0;
      ++seen;
    }
  }
  atomicAdd(&s_in_order, in_order);
  atomicAdd(&s_seen, seen);
  __syncthreads();
  if (threadIdx.x == 0) *flag = (s_seen > 0 && 2 * s_in_order >= s_seen) ? 1 : 0;
}

cudaError_t launch_page_order(const AttnArgs& a, int32_t* flag, cudaStream_t stream) {
  if (a.geom.page_tokens > 32) return cudaErrorInvalidValue;
  page_order_kernel<<<1, 256, 0, stream>>>(a.slots, a.lens, a.batch, a.geom, flag);
  return cudaGetLastError();
}

}  // namespace echokv
