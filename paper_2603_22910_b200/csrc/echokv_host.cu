// C-ABI of the EchoKV library: argument checking, workspace layout, kernel selection.
// All device memory belongs to the caller; nothing here allocates on the device.
#include <cmath>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "kernels.h"
#include "recon_tc.h"
#include "stored_mma.h"
#include "absorbed.h"
#include "prefill.h"

using namespace echokv;

namespace {

constexpr uint64_t kAlign = 256;
inline uint64_t align_up(uint64_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Derived {
  int D, m, d_in, d_drop, g, elem, part_tokens, capacity, max_parts;
  int mk;              // K dims a compressed layer stores: m, or D in the "save K" setting
  bool save_k;
  bool head_aligned;   // m ends on a head boundary
  // Where m splits a head the explicit kernels treat that head as predicted: m_heads = flat dims of the whole
  // retained heads, split = m - m_heads stored dims of the split head, which predictors extended by `split`
  // one-hot rows pass through.  The extended predictors (and biases) of every compressed layer live in the workspace.
  int m_heads, split;
  uint64_t wx_bytes, bx_bytes;   // one extended predictor / bias (256-byte multiples), 0 when m is head-aligned
  uint64_t off_status, off_ml, off_o, off_q, off_k, off_v, off_out, off_lens, off_pos, off_wx, total;
};

int derive(const echokv_config* c, Derived* d) {
  if (!c) return ECHOKV_EINVAL;
  if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->group_size < 1 ||
      c->max_batch < 1 || c->max_pages_per_seq < 1 || c->n_pages < 1)
    return ECHOKV_EINVAL;
  if (c->n_q_heads % c->n_kv_heads != 0) return ECHOKV_EINVAL;
  if (c->n_retained_heads < 0 || c->n_retained_heads > c->n_kv_heads) return ECHOKV_EINVAL;
  if (c->dtype != ECHOKV_BF16 && c->dtype != ECHOKV_FP32) return ECHOKV_EINVAL;
  if (!(c->softmax_scale >= 0.f) || !std::isfinite(c->softmax_scale)) return ECHOKV_EINVAL;
  if (c->head_dim != 64 && c->head_dim != 128) return ECHOKV_EUNSUPPORTED;
  if (c->page_tokens != 16 && c->page_tokens != 32 && c->page_tokens != 64 && c->page_tokens != 128)
    return ECHOKV_EUNSUPPORTED;
  d->g = c->n_q_heads / c->n_kv_heads;
  if (d->g != 1 && d->g != 2 && d->g != 4 && d->g != 8) return ECHOKV_EUNSUPPORTED;
  const long long cap = (long long)c->max_pages_per_seq * c->page_tokens;
  if (cap > (1ll << 30)) return ECHOKV_EINVAL;
  d->D = c->n_kv_heads * c->head_dim;
  d->m = c->n_retained_heads * c->head_dim;
  if (c->n_retained_dims != 0) {
    // m given in flat dims (the paper's m = 64: half of the first head): any multiple of 64 up to D
    if (c->n_retained_dims < 0 || c->n_retained_dims > d->D) return ECHOKV_EINVAL;
    if (c->n_retained_dims % 64 != 0) return ECHOKV_EUNSUPPORTED;
    d->m = c->n_retained_dims;
  }
  d->head_aligned = d->m % c->head_dim == 0;
  d->m_heads = d->m / c->head_dim * c->head_dim;
  d->split = d->m - d->m_heads;
  d->save_k = c->save_k != 0 && d->m < d->D;
  d->mk = d->save_k ? d->D : d->m;
  d->d_in = d->D + d->m;
  d->d_drop = d->D - d->m;
  d->elem = c->dtype == ECHOKV_BF16 ? 2 : 4;
  d->part_tokens = (c->dtype == ECHOKV_BF16 && c->head_dim == 128) ? kPairPartTokens : kSimtTileTokens;
  d->capacity = (int)cap;
  d->max_parts = (d->capacity + d->part_tokens - 1) / d->part_tokens + 1;   // + the sink / window partial
  uint64_t off = 0;
  d->off_status = off; off += kAlign;
  const uint64_t n_part = (uint64_t)c->max_batch * c->n_q_heads * d->max_parts;
  d->off_ml = off; off = align_up(off + n_part * sizeof(float2));
  d->off_o = off; off = align_up(off + n_part * c->head_dim * sizeof(float));
  const uint64_t q_bytes = (uint64_t)c->max_batch * c->n_q_heads * c->head_dim * d->elem;
  const uint64_t kv_bytes = (uint64_t)c->max_batch * d->D * d->elem;
  d->off_q = off; off = align_up(off + q_bytes);
  d->off_k = off; off = align_up(off + kv_bytes);
  d->off_v = off; off = align_up(off + kv_bytes);
  d->off_out = off; off = align_up(off + (uint64_t)c->max_batch * c->n_q_heads * c->head_dim * 4);
  d->off_lens = off; off = align_up(off + (uint64_t)c->max_batch * 4);
  d->off_pos = off; off = align_up(off + (uint64_t)c->max_batch * 4);
  d->off_wx = off;
  d->wx_bytes = d->bx_bytes = 0;
  if (d->split > 0) {
    d->wx_bytes = align_up((uint64_t)(d->D - d->m_heads) * d->d_in * d->elem);
    d->bx_bytes = align_up((uint64_t)(d->D - d->m_heads) * d->elem);
    off += (uint64_t)c->n_layers * 2 * (d->wx_bytes + d->bx_bytes);     // K and V of every layer
  }
  d->total = off;
  return ECHOKV_OK;
}

struct Layer {
  void* k_pool = nullptr;
  void* v_pool = nullptr;
  const void* Wk = nullptr;
  const void* Wv = nullptr;
  const void* bk = nullptr;
  const void* bv = nullptr;
  // what the explicit kernels read: the predictors as given, or (m splits a head) their extended copies
  const void* Wk_x = nullptr;
  const void* Wv_x = nullptr;
  const void* bk_x = nullptr;
  const void* bv_x = nullptr;
  bool anchor = false;
  void* k_side = nullptr;   // dropped dims of the sink and recent-window tokens (compressed layers)
  void* v_side = nullptr;
  TcLayerMaps tc;     // tensor maps of the tensor-core path (valid when tc.ready)
  CUtensorMap stored_k, stored_v;   // tensor maps of the stored-head kernel (valid when ctx.stored_path == 1)
  CUtensorMap stored_k_run, stored_v_run;   // the same pools in boxes of 64 token rows
};

}  // namespace

struct echokv_ctx {
  echokv_config cfg;
  Derived d;
  std::vector<Layer> layers;
  const int32_t* table = nullptr;
  unsigned char* ws = nullptr;
  int sm_count = 0;
  int path = 0;          // see echokv_decode_path
  bool tc_capable = false;
  int n_sink = 0, n_window = 0;   // tokens kept at full precision (0, 0 = none)
  RopeTable rope;                 // rotate-on-read of un-rotated cached keys (off while rope.cs is null)
  bool absorbed_capable = false;  // shape served by the absorbed-predictor kernels
  int decode_mode = 0;            // 0 = explicit reconstruction (Eq. 3, 6, 7 as written), 1 = absorbed predictors
  unsigned char* ws_absorbed = nullptr;
  AbsorbLayout alay;
  AbsorbMaps amaps;
  bool stored_capable = false;   // shape served by the TMA + mma.sync stored-head kernel
  int stored_path = 0;           // 0 = CUDA-core kernel, 1 = TMA + mma.sync kernel
  int64_t launches = 0;
  float scale = 0.f;
  std::vector<int32_t> pos_scratch;
  bool timing = false;
  size_t timed = 0;                                         // event pairs in use
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> events;  // grown on demand, reused
  std::vector<int> event_kind;                              // ECHOKV_TIMED_* of each pair
  ~echokv_ctx() {
    for (auto& e : events) {
      cudaEventDestroy(e.first);
      cudaEventDestroy(e.second);
    }
  }
};

namespace {

int32_t* status_ptr(echokv_ctx* c) { return reinterpret_cast<int32_t*>(c->ws + c->d.off_status); }
// item sizes the stored-head kernel publishes for the merge kernel: kStoredMaxLaunches words that
// share the status word's 256-byte block
int32_t* item_tokens_ptr(echokv_ctx* c) { return reinterpret_cast<int32_t*>(c->ws + c->d.off_status + 64); }
// the word the page-order kernel writes (decode path 5)
int32_t* page_order_ptr(echokv_ctx* c) { return reinterpret_cast<int32_t*>(c->ws + c->d.off_status + 32); }

PageGeom geom_of(const echokv_ctx* c) {
  PageGeom g;
  g.table = c->table;
  g.max_batch = c->cfg.max_batch;
  g.max_pages_per_seq = c->cfg.max_pages_per_seq;
  g.page_tokens = c->cfg.page_tokens;
  g.n_pages = c->cfg.n_pages;
  return g;
}

AttnArgs attn_args(echokv_ctx* c, const void* q, const int32_t* slots, const int32_t* lens, int B) {
  AttnArgs a;
  a.dtype = c->cfg.dtype;
  a.n_q_heads = c->cfg.n_q_heads;
  a.n_kv_heads = c->cfg.n_kv_heads;
  a.head_dim = c->cfg.head_dim;
  a.batch = B;
  a.scale_log2e = c->scale * kLog2e;
  a.q = q;
  a.slots = slots;
  a.lens = lens;
  a.geom = geom_of(c);
  a.parts.ml = reinterpret_cast<float2*>(c->ws + c->d.off_ml);
  a.parts.o = reinterpret_cast<float*>(c->ws + c->d.off_o);
  a.parts.max_parts = c->d.max_parts;
  a.status = status_ptr(c);
  a.rope = c->rope;
  return a;
}

int stored_splits(const echokv_ctx* c, int B, int n_heads) {
  if (n_heads <= 0) return 1;
  const int ctas = B * n_heads;
  int n = (4 * c->sm_count + ctas - 1) / ctas;
  if (n > c->d.max_parts) n = c->d.max_parts;
  if (n > c->cfg.max_pages_per_seq) n = c->cfg.max_pages_per_seq;
  if (n < 1) n = 1;
  return n;
}

// Event pair around the dominant kernel of a call (only while timing is enabled).
struct ScopedKernelTimer {
  echokv_ctx* c;
  cudaStream_t s;
  cudaEvent_t stop = nullptr;
  ScopedKernelTimer(echokv_ctx* ctx, cudaStream_t stream, int kind) : c(ctx), s(stream) {
    if (!c->timing) return;
    if (c->timed == c->events.size()) {
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess) return;
      if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return; }
      c->events.emplace_back(a, b);
      c->event_kind.push_back(kind);
    }
    c->event_kind[c->timed] = kind;
    auto& e = c->events[c->timed++];
    cudaEventRecord(e.first, s);
    stop = e.second;
  }
  ~ScopedKernelTimer() {
    if (stop) cudaEventRecord(stop, s);
  }
};

// An event pair of the given kind for a kernel the callee launches itself (null while timing is off).
bool timed_pair(echokv_ctx* c, int kind, cudaEvent_t* start, cudaEvent_t* stop) {
  if (!c->timing) return false;
  if (c->timed == c->events.size()) {
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess) return false;
    if (cudaEventCreate(&b) != cudaSuccess) { cudaEventDestroy(a); return false; }
    c->events.emplace_back(a, b);
    c->event_kind.push_back(kind);
  }
  c->event_kind[c->timed] = kind;
  *start = c->events[c->timed].first;
  *stop = c->events[c->timed].second;
  ++c->timed;
  return true;
}

bool side_active(const echokv_ctx* c, const Layer& L) {
  return !L.anchor && c->d.d_drop > 0 && (c->n_sink > 0 || c->n_window > 0);
}

SideArgs side_args(const echokv_ctx* c, const Layer& L) {
  SideArgs s;
  s.k_side = L.k_side; s.v_side = L.v_side;
  s.n_sink = c->n_sink; s.n_window = c->n_window; s.d_drop = c->d.d_drop;
  return s;
}

// The new token's dropped dims of a compressed layer go to the side buffers while a sink / window is set.
int append_side(echokv_ctx* c, const Layer& L, const void* k_new, const void* v_new, const int32_t* slots,
                const int32_t* positions, int B, int n_tokens, cudaStream_t s) {
  if (!side_active(c, L)) return ECHOKV_OK;
  if (launch_append_side(c->cfg.dtype, side_args(c, L), c->d.m, c->d.D, k_new, v_new, slots, positions, B, n_tokens,
                         c->cfg.max_batch, status_ptr(c), s) != cudaSuccess)
    return ECHOKV_ECUDA;
  c->launches += 1;
  return ECHOKV_OK;
}

// The kernels read queries and new K / V rows with 16-byte loads and may store results 16 bytes at a time.
inline bool aligned16(const void* p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

int check_call(echokv_ctx* c, int layer, const void* q, const float* out, const int32_t* lens, int B) {
  if (!c || !q || !out || !lens) return ECHOKV_EINVAL;
  if (!aligned16(q) || !aligned16(out)) return ECHOKV_EINVAL;
  if (layer < 0 || layer >= c->cfg.n_layers || B < 1) return ECHOKV_EINVAL;
  if (B > c->cfg.max_batch) return ECHOKV_ECAPACITY;
  if (!c->table) return ECHOKV_ENOTABLE;
  return ECHOKV_OK;
}

// Eq. 7 for the stored KV heads 0 .. n_heads-1 of layer L (pool row width `width`), as split-K
// partials.  *item_tokens receives the device array the merge kernel reads the partial count
// from (null: n_splits partials per head).
cudaError_t attend_stored_heads(echokv_ctx* c, const AttnArgs& a, const Layer& L, int width, int n_heads,
                                int n_splits, const int32_t** item_tokens, cudaStream_t s) {
  *item_tokens = nullptr;
  if (n_heads == 0) return cudaSuccess;
  c->launches += 1;
  if (c->stored_path == 1) {
    *item_tokens = item_tokens_ptr(c);
    return launch_attn_stored_mma(a, L.stored_k, L.stored_v, L.stored_k_run, L.stored_v_run, n_heads,
                                  item_tokens_ptr(c), c->sm_count, s);
  }
  return launch_attn_stored(a, L.k_pool, L.v_pool, width, n_heads, n_splits, s);
}

int attend_stored_layer(echokv_ctx* c, const Layer& L, const void* q, float* out,
                        const int32_t* slots, const int32_t* lens, int B, cudaStream_t s) {
  AttnArgs a = attn_args(c, q, slots, lens, B);
  const int H = c->cfg.n_kv_heads;
  const int n_splits = stored_splits(c, B, H);
  const int32_t* item_tokens = nullptr;
  {
    ScopedKernelTimer timer(c, s, ECHOKV_TIMED_STORED);
    if (attend_stored_heads(c, a, L, c->d.D, H, n_splits, &item_tokens, s) != cudaSuccess) return ECHOKV_ECUDA;
  }
  if (launch_merge(a, out, H, n_splits, item_tokens, kStoredMaxBatchPerLaunch, c->d.part_tokens, nullptr, s) !=
      cudaSuccess)
    return ECHOKV_ECUDA;
  c->launches += 1;
  return ECHOKV_OK;
}

}  // namespace

extern "C" {

int echokv_query_sizes(const echokv_config* cfg, echokv_sizes* out) {
  if (!out) return ECHOKV_EINVAL;
  Derived d;
  const int rc = derive(cfg, &d);
  if (rc != ECHOKV_OK) return rc;
  const uint64_t rows = (uint64_t)cfg->n_pages * cfg->page_tokens;
  out->anchor_pool_bytes = rows * d.D * d.elem;
  out->compressed_pool_bytes = rows * d.m * d.elem;
  out->block_table_bytes = (uint64_t)cfg->max_batch * cfg->max_pages_per_seq * 4;
  out->workspace_bytes = d.total;
  out->max_partials = d.max_parts;
  out->reserved = 0;
  return ECHOKV_OK;
}

int echokv_create(const echokv_config* cfg, const echokv_buffers* buf, echokv_ctx** out) {
  if (!out) return ECHOKV_EINVAL;
  *out = nullptr;
  Derived d;
  int rc = derive(cfg, &d);
  if (rc != ECHOKV_OK) return rc;
  if (!buf || !buf->k_pools || !buf->v_pools || !buf->workspace) return ECHOKV_EINVAL;
  if (buf->workspace_bytes < d.total) return ECHOKV_ECAPACITY;
  if (reinterpret_cast<uintptr_t>(buf->workspace) % kAlign != 0) return ECHOKV_EINVAL;
  for (int l = 0; l < cfg->n_layers; ++l) {
    const bool anchor = l % cfg->group_size == 0;
    const bool needs_k = anchor || d.mk > 0, needs_v = anchor || d.m > 0;
    if ((needs_k && !buf->k_pools[l]) || (needs_v && !buf->v_pools[l])) return ECHOKV_EINVAL;
    if ((needs_k && reinterpret_cast<uintptr_t>(buf->k_pools[l]) % 16 != 0) ||
        (needs_v && reinterpret_cast<uintptr_t>(buf->v_pools[l]) % 16 != 0))
      return ECHOKV_EINVAL;
  }
  echokv_ctx* c = new (std::nothrow) echokv_ctx();
  if (!c) return ECHOKV_EINVAL;
  c->cfg = *cfg;
  c->d = d;
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
  c->ws = static_cast<unsigned char*>(buf->workspace);
  c->layers.resize(cfg->n_layers);
  bool any_compressed = false;
  for (int l = 0; l < cfg->n_layers; ++l) {
    c->layers[l].anchor = l % cfg->group_size == 0;
    c->layers[l].k_pool = buf->k_pools[l];
    c->layers[l].v_pool = buf->v_pools[l];
    any_compressed |= !c->layers[l].anchor;
  }
  if (cudaSetDevice(cfg->device) != cudaSuccess) { delete c; return ECHOKV_ECUDA; }
  if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess) {
    delete c;
    return ECHOKV_ECUDA;
  }
  if (cudaMemset(c->ws + d.off_status, 0, kAlign) != cudaSuccess) { delete c; return ECHOKV_ECUDA; }
  c->tc_capable = tc_shape_supported(cfg->dtype, cfg->head_dim, cfg->page_tokens, d.D, d.m);
  if (!any_compressed || d.d_drop == 0) c->path = 0;
  else if (d.save_k) {
    // keys kept whole: served by the absorbed mode only
    if (!absorbed_supported(cfg->dtype, cfg->head_dim, cfg->n_q_heads, cfg->n_kv_heads, d.m, cfg->page_tokens)) {
      delete c;
      return ECHOKV_EUNSUPPORTED;
    }
    c->path = 0;
  }
  else if (!c->tc_capable) c->path = 1;
  else {
    // Long contractions (many 64-feature chunks per phase, few query heads per KV head) hide the
    // epilogue by themselves and run best with all of tensor memory given to one phase; short ones need the
    // CTA-pair kernel's double-buffered accumulators.  Of the two kernels for long contractions the one-CTA kernel
    // is the faster while the pages of a tile follow one another in the pool (fewer, taller TMA boxes), but with
    // small pages in no particular order -- what a paged pool becomes in service -- it is bound by the number of
    // copies per stage; the four-heads-per-pair kernel needs half as many and is indifferent to the order
    // (measured at the 7B layer shape, 16-token pages: in order 2.08 against 2.28 ms, random order 2.34-2.42
    // against 2.28 ms).  So small pages go to the latter.
    const int chunks = d.d_in / 64;
    if (chunks <= 12 * d.g) c->path = 3;
    else c->path = (recon_quad_supported(d.g) && cfg->page_tokens <= 32) ? 5 : 2;
  }
  if (c->tc_capable) {
    // tensor maps of every pool (the predictors' maps follow in echokv_set_weights)
    for (int l = 0; l < cfg->n_layers; ++l) {
      Layer& L = c->layers[l];
      const int k_width = L.anchor ? d.D : d.mk, v_width = L.anchor ? d.D : d.m;
      if (k_width == 0 && v_width == 0) continue;
      const cudaError_t e = tc_encode_pool_maps(&L.tc, L.k_pool, k_width, L.v_pool, v_width,
                                                (uint64_t)cfg->n_pages * cfg->page_tokens,
                                                cfg->page_tokens);
      if (e != cudaSuccess) { delete c; return ECHOKV_ECUDA; }
    }
  }
  c->stored_capable = stored_mma_supported(cfg->dtype, cfg->head_dim, d.g, cfg->max_batch);
  if (c->stored_capable) {
    const int box_rows = stored_rows_per_box(cfg->page_tokens);
    for (int l = 0; l < cfg->n_layers; ++l) {
      Layer& L = c->layers[l];
      const int width = L.anchor ? d.D : d.m;
      const uint64_t rows = (uint64_t)cfg->n_pages * cfg->page_tokens;
      if (!L.anchor && d.save_k) {
        // keys kept whole: no stored-head attention on that layer, but its keys are scored from the pool when a
        // rotation is set (the K maps only)
        if (encode_pool_group_map(&L.stored_k, L.k_pool, d.D, rows, box_rows) != cudaSuccess ||
            encode_pool_group_map(&L.stored_k_run, L.k_pool, d.D, rows, 64) != cudaSuccess) {
          delete c;
          return ECHOKV_ECUDA;
        }
        continue;
      }
      if (width == 0) continue;
      if (encode_pool_group_map(&L.stored_k, L.k_pool, width, rows, box_rows) != cudaSuccess ||
          encode_pool_group_map(&L.stored_v, L.v_pool, width, rows, box_rows) != cudaSuccess ||
          encode_pool_group_map(&L.stored_k_run, L.k_pool, width, rows, 64) != cudaSuccess ||
          encode_pool_group_map(&L.stored_v_run, L.v_pool, width, rows, 64) != cudaSuccess) {
        delete c;
        return ECHOKV_ECUDA;
      }
    }
    c->stored_path = 1;
  }
  *out = c;
  return ECHOKV_OK;
}

void echokv_destroy(echokv_ctx* ctx) { delete ctx; }

int echokv_set_weights(echokv_ctx* c, int layer, const void* Wk, const void* Wv, const void* bk,
                       const void* bv) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return ECHOKV_EINVAL;
  Layer& L = c->layers[layer];
  if (L.anchor) return ECHOKV_ENOTCOMPRESSED;
  if (c->d.d_drop > 0 && (!Wv || (!Wk && !c->d.save_k))) return ECHOKV_EINVAL;   // (keys kept whole: no K predictor)
  if ((reinterpret_cast<uintptr_t>(Wk) | reinterpret_cast<uintptr_t>(Wv)) % 16 != 0) return ECHOKV_EINVAL;
  L.Wk = Wk; L.Wv = Wv; L.bk = bk; L.bv = bv;
  L.Wk_x = Wk; L.Wv_x = Wv; L.bk_x = bk; L.bv_x = bv;
  const Derived& d = c->d;
  if (d.split > 0 && d.d_drop > 0) {
    // m splits a head: build the extended predictors in the workspace (device work on the default stream, waited for)
    if (cudaSetDevice(c->cfg.device) != cudaSuccess) return ECHOKV_ECUDA;
    unsigned char* base = c->ws + d.off_wx + (uint64_t)layer * 2 * (d.wx_bytes + d.bx_bytes);
    void* wkx = base; void* wvx = base + d.wx_bytes;
    void* bkx = base + 2 * d.wx_bytes; void* bvx = base + 2 * d.wx_bytes + d.bx_bytes;
    const int pass_col0 = d.D + d.m_heads;            // input column of local dim m_heads
    if (Wk && launch_extend_predictor(c->cfg.dtype, Wk, bk, wkx, bkx, d.d_drop, d.d_in, d.split, pass_col0, nullptr) !=
                  cudaSuccess)
      return ECHOKV_ECUDA;
    if (launch_extend_predictor(c->cfg.dtype, Wv, bv, wvx, bvx, d.d_drop, d.d_in, d.split, pass_col0, nullptr) !=
        cudaSuccess)
      return ECHOKV_ECUDA;
    if (cudaStreamSynchronize(nullptr) != cudaSuccess) return ECHOKV_ECUDA;
    c->launches += Wk ? 2 : 1;
    L.Wk_x = Wk ? wkx : nullptr; L.Wv_x = wvx;
    L.bk_x = (Wk && bk) ? bkx : nullptr; L.bv_x = bv ? bvx : nullptr;
  }
  if (c->tc_capable && d.d_drop > 0) {
    if (tc_encode_weight_maps(&L.tc, L.Wk_x, L.Wv_x, d.D - d.m_heads, d.d_in) != cudaSuccess) return ECHOKV_ECUDA;
  }
  return ECHOKV_OK;
}

int echokv_set_block_table(echokv_ctx* c, const int32_t* dev_block_table) {
  if (!c || !dev_block_table) return ECHOKV_EINVAL;
  c->table = dev_block_table;
  return ECHOKV_OK;
}

int echokv_set_decode_path(echokv_ctx* c, int path) {
  if (!c) return ECHOKV_EINVAL;
  if (c->path == 0) return path == 0 ? ECHOKV_OK : ECHOKV_EINVAL;
  if (path == 1) { c->path = 1; return ECHOKV_OK; }
  if (path >= 2 && path <= 5) {
    if (!c->tc_capable || (path >= 4 && !recon_quad_supported(c->d.g))) return ECHOKV_EUNSUPPORTED;
    if (path == 5 && c->cfg.page_tokens > 32) return ECHOKV_EUNSUPPORTED;
    c->path = path;
    return ECHOKV_OK;
  }
  return ECHOKV_EINVAL;
}

int echokv_side_buffer_bytes(const echokv_config* cfg, int n_sink, int n_window, uint64_t* out) {
  if (!out || n_sink < 0 || n_window < 0) return ECHOKV_EINVAL;
  Derived d;
  const int rc = derive(cfg, &d);
  if (rc != ECHOKV_OK) return rc;
  if (n_sink + n_window > 4096) return ECHOKV_EUNSUPPORTED;
  *out = (uint64_t)cfg->max_batch * (uint64_t)(n_sink + n_window) * d.d_drop * d.elem;
  return ECHOKV_OK;
}

int echokv_set_full_precision_window(echokv_ctx* c, int n_sink, int n_window, void* const* k_side,
                                     void* const* v_side) {
  if (!c || n_sink < 0 || n_window < 0) return ECHOKV_EINVAL;
  if (n_sink + n_window > 4096) return ECHOKV_EUNSUPPORTED;
  const bool on = (n_sink > 0 || n_window > 0) && c->d.d_drop > 0;
  const bool need_k = !c->d.save_k;     // (keys kept whole are in the pool already: no K side buffer is read or written)
  if (on) {
    if (!v_side || (need_k && !k_side)) return ECHOKV_EINVAL;
    for (int l = 0; l < c->cfg.n_layers; ++l) {
      if (c->layers[l].anchor) continue;
      if (!v_side[l] || (need_k && !k_side[l])) return ECHOKV_EINVAL;
      if ((reinterpret_cast<uintptr_t>(need_k ? k_side[l] : nullptr) | reinterpret_cast<uintptr_t>(v_side[l])) % 16 != 0)
        return ECHOKV_EINVAL;
    }
    for (int l = 0; l < c->cfg.n_layers; ++l) {
      c->layers[l].k_side = (c->layers[l].anchor || !need_k) ? nullptr : k_side[l];
      c->layers[l].v_side = c->layers[l].anchor ? nullptr : v_side[l];
    }
  }
  c->n_sink = on ? n_sink : 0;
  c->n_window = on ? n_window : 0;
  return ECHOKV_OK;
}

int echokv_rope_table_bytes(const echokv_config* cfg, uint64_t* out) {
  if (!out) return ECHOKV_EINVAL;
  Derived d;
  const int rc = derive(cfg, &d);
  if (rc != ECHOKV_OK) return rc;
  *out = (uint64_t)rope_table_pairs(d.capacity, cfg->head_dim) * sizeof(float2);
  return ECHOKV_OK;
}

int echokv_set_rope(echokv_ctx* c, double theta, void* table, uint64_t table_bytes, void* stream) {
  if (!c) return ECHOKV_EINVAL;
  if (table == nullptr || !(theta > 0.0)) {      // off
    if (table != nullptr || theta != 0.0) return ECHOKV_EINVAL;
    c->rope = RopeTable();
    return ECHOKV_OK;
  }
  if (!std::isfinite(theta) || theta < 1.0) return ECHOKV_EINVAL;
  // (a rotation that depends on the token cannot be folded into the queries: the K side is then explicit, the
  // tensor-core kernels for the predicted heads and the stored-head kernels for the rest)
  if (!c->d.head_aligned && !c->d.save_k && !c->tc_capable) return ECHOKV_EUNSUPPORTED;
  uint64_t need = 0;
  const int rc = echokv_rope_table_bytes(&c->cfg, &need);
  if (rc != ECHOKV_OK) return rc;
  if (table_bytes < need) return ECHOKV_ECAPACITY;
  if (reinterpret_cast<uintptr_t>(table) % 16 != 0) return ECHOKV_EINVAL;
  if (launch_rope_table(static_cast<float2*>(table), c->d.capacity, c->cfg.head_dim, theta,
                        static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return ECHOKV_ECUDA;
  c->launches += 3;
  c->rope = rope_table_view(static_cast<const float2*>(table), c->d.capacity, c->cfg.head_dim);
  return ECHOKV_OK;
}

int echokv_rope_enabled(const echokv_ctx* c) { return c && c->rope.cs != nullptr ? 1 : 0; }

int echokv_absorbed_workspace_bytes(const echokv_config* cfg, uint64_t* out) {
  if (!out) return ECHOKV_EINVAL;
  Derived d;
  const int rc = derive(cfg, &d);
  if (rc != ECHOKV_OK) return rc;
  if (!absorbed_supported(cfg->dtype, cfg->head_dim, cfg->n_q_heads, cfg->n_kv_heads, d.m, cfg->page_tokens) ||
      cfg->max_batch > 256)
    return ECHOKV_EUNSUPPORTED;
  AbsorbLayout lay;
  absorbed_layout(cfg->max_batch, cfg->n_q_heads, d.d_in, d.capacity, &lay);
  *out = lay.total;
  return ECHOKV_OK;
}

int echokv_enable_absorbed(echokv_ctx* c, void* workspace, uint64_t workspace_bytes) {
  if (!c || !workspace) return ECHOKV_EINVAL;
  uint64_t need = 0;
  const int rc = echokv_absorbed_workspace_bytes(&c->cfg, &need);
  if (rc != ECHOKV_OK) return rc;
  if (!c->tc_capable) return ECHOKV_EUNSUPPORTED;
  if (workspace_bytes < need) return ECHOKV_ECAPACITY;
  if (reinterpret_cast<uintptr_t>(workspace) % kAlign != 0) return ECHOKV_EINVAL;
  c->ws_absorbed = static_cast<unsigned char*>(workspace);
  absorbed_layout(c->cfg.max_batch, c->cfg.n_q_heads, c->d.d_in, c->d.capacity, &c->alay);
  if (absorbed_encode_maps(&c->amaps, c->ws_absorbed, c->alay, c->cfg.max_batch, c->d.d_in) != cudaSuccess)
    return ECHOKV_ECUDA;
  c->absorbed_capable = true;
  c->decode_mode = 1;
  return ECHOKV_OK;
}

int echokv_decode_mode(const echokv_ctx* c) { return c ? c->decode_mode : 0; }

int echokv_set_decode_mode(echokv_ctx* c, int mode) {
  if (!c || (mode != 0 && mode != 1)) return ECHOKV_EINVAL;
  if (mode == 1 && !c->absorbed_capable) return ECHOKV_EUNSUPPORTED;
  c->decode_mode = mode;
  return ECHOKV_OK;
}

int echokv_stored_path(const echokv_ctx* c) { return c ? c->stored_path : 0; }

int echokv_set_stored_path(echokv_ctx* c, int path) {
  if (!c || (path != 0 && path != 1)) return ECHOKV_EINVAL;
  if (path == 1 && !c->stored_capable) return ECHOKV_EUNSUPPORTED;
  c->stored_path = path;
  return ECHOKV_OK;
}

int echokv_append_kv_chunk(echokv_ctx* c, int layer, const void* k_new, const void* v_new,
                           const int32_t* dev_seq_slots, const int32_t* dev_first_positions, int n_tokens, int B,
                           void* stream) {
  if (!c || !k_new || !v_new || !dev_first_positions) return ECHOKV_EINVAL;
  if (!aligned16(k_new) || !aligned16(v_new)) return ECHOKV_EINVAL;
  if (layer < 0 || layer >= c->cfg.n_layers || B < 1 || n_tokens < 1) return ECHOKV_EINVAL;
  if (B > c->cfg.max_batch || n_tokens > c->d.capacity || n_tokens > 65535) return ECHOKV_ECAPACITY;
  if (!c->table) return ECHOKV_ENOTABLE;
  const Layer& L = c->layers[layer];
  const int k_width = L.anchor ? c->d.D : c->d.mk, v_width = L.anchor ? c->d.D : c->d.m;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (k_width == 0 && v_width == 0)   // nothing of this layer is kept in the pools (m = 0)
    return append_side(c, L, k_new, v_new, dev_seq_slots, dev_first_positions, B, n_tokens, s);
  const cudaError_t e = launch_append(c->cfg.dtype, L.k_pool, L.v_pool, k_width, v_width, c->d.D, k_new, v_new,
                                      dev_seq_slots, dev_first_positions, B, n_tokens, geom_of(c), status_ptr(c), s);
  if (e != cudaSuccess) return ECHOKV_ECUDA;
  c->launches += 1;
  return append_side(c, L, k_new, v_new, dev_seq_slots, dev_first_positions, B, n_tokens, s);
}

int echokv_append_kv(echokv_ctx* c, int layer, const void* k_new, const void* v_new,
                     const int32_t* dev_seq_slots, const int32_t* dev_positions, int B, void* stream) {
  return echokv_append_kv_chunk(c, layer, k_new, v_new, dev_seq_slots, dev_positions, 1, B, stream);
}

int echokv_compress_layer(echokv_ctx* c, int layer, const void* k_full, const void* v_full,
                          const int32_t* dev_seq_slots, const int32_t* dev_seq_begins,
                          const int32_t* dev_seq_lens, int B, void* stream) {
  if (!c || !k_full || !v_full || !dev_seq_lens) return ECHOKV_EINVAL;
  if (layer < 0 || layer >= c->cfg.n_layers || B < 1) return ECHOKV_EINVAL;
  if ((reinterpret_cast<uintptr_t>(k_full) | reinterpret_cast<uintptr_t>(v_full)) % 16 != 0) return ECHOKV_EINVAL;
  if (B > c->cfg.max_batch) return ECHOKV_ECAPACITY;
  if (!c->table) return ECHOKV_ENOTABLE;
  const Layer& L = c->layers[layer];
  if (L.anchor) return ECHOKV_ENOTCOMPRESSED;
  const bool side = side_active(c, L);
  if (c->d.mk == 0 && !side) return ECHOKV_OK;         // nothing of this layer is kept
  const SideArgs sa = side_args(c, L);
  if (launch_compress(c->d.elem, k_full, v_full, L.k_pool, L.v_pool, side ? &sa : nullptr, c->d.D, c->d.mk, c->d.m,
                      dev_seq_slots, dev_seq_begins, dev_seq_lens, B, geom_of(c), status_ptr(c),
                      static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return ECHOKV_ECUDA;
  c->launches += 1;
  return ECHOKV_OK;
}

int echokv_prefill_scratch_bytes(const echokv_config* cfg, uint64_t* out) {
  if (!out) return ECHOKV_EINVAL;
  Derived d;
  const int rc = derive(cfg, &d);
  if (rc != ECHOKV_OK) return rc;
  if (cfg->dtype != ECHOKV_BF16 || cfg->head_dim != 128) return ECHOKV_EUNSUPPORTED;
  // K~ rows, V~ rows, and one fp32 per (sequence, query, query head) for the sink / window combination
  *out = 2ull * (uint64_t)cfg->max_batch * (uint64_t)d.capacity * (uint64_t)d.D * 2ull +
         (uint64_t)cfg->max_batch * (uint64_t)d.capacity * (uint64_t)cfg->n_q_heads * 4ull;
  return ECHOKV_OK;
}

int echokv_prefill_attention(echokv_ctx* c, int layer, const void* q, float* out, int n_q,
                             const int32_t* dev_seq_slots, const int32_t* dev_seq_lens, int B,
                             const void* k_recent, const void* v_recent,
                             void* scratch, uint64_t scratch_bytes, void* stream) {
  const int rc = check_call(c, layer, q, out, dev_seq_lens, B);
  if (rc != ECHOKV_OK) return rc;
  if (!scratch || n_q < 1 || reinterpret_cast<uintptr_t>(scratch) % 16 != 0) return ECHOKV_EINVAL;
  const Layer& L = c->layers[layer];
  const bool compressed = !L.anchor && c->d.d_drop > 0;
  if (c->cfg.dtype != ECHOKV_BF16 || c->cfg.head_dim != 128) return ECHOKV_EUNSUPPORTED;
  if (compressed && !c->tc_capable) return ECHOKV_EUNSUPPORTED;
  const bool windowed = compressed && side_active(c, L);
  if (windowed && (!k_recent || !v_recent || !aligned16(k_recent) || !aligned16(v_recent))) return ECHOKV_EINVAL;
  const bool keys_whole = compressed && c->d.save_k;      // Section 5.2: nothing to predict on the K side
  if (n_q > c->d.capacity) return ECHOKV_ECAPACITY;
  const uint64_t rows_bytes = (uint64_t)B * c->d.capacity * c->d.D * 2ull;     // one of K~, V~
  const uint64_t lse_bytes = (uint64_t)B * n_q * c->cfg.n_q_heads * 4ull;
  if (scratch_bytes < 2 * rows_bytes + (windowed ? lse_bytes : 0)) return ECHOKV_ECAPACITY;
  if (compressed && (!L.Wv || (!L.Wk && !keys_whole))) return ECHOKV_ENOWEIGHTS;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  AttnArgs a = attn_args(c, q, dev_seq_slots, dev_seq_lens, B);
  __nv_bfloat16* k_rows = static_cast<__nv_bfloat16*>(scratch);
  __nv_bfloat16* v_rows = k_rows + rows_bytes / 2;
  const int k_width = compressed ? c->d.mk : c->d.D, v_width = compressed ? c->d.m : c->d.D;
  // stored dims as they are (keys rotated to their positions), then the predicted ones beside them; of a head that m
  // splits nothing is copied here: the extended predictor writes it whole (a rotation needs both halves of a head)
  const int k_copy = (compressed && !keys_whole) ? c->d.m_heads : k_width;
  const int v_copy = compressed ? c->d.m_heads : v_width;
  if (launch_gather_rows(a, L.k_pool, k_width, k_copy, k_rows, c->d.capacity, c->d.D, true, 0, s) != cudaSuccess ||
      launch_gather_rows(a, L.v_pool, v_width, v_copy, v_rows, c->d.capacity, c->d.D, false, 128, s, true) != cudaSuccess)
    return ECHOKV_ECUDA;
  c->launches += (k_copy > 0 ? 1 : 0) + 1;
  if (compressed) {
    const Layer& A = c->layers[layer - layer % c->cfg.group_size];
    ReconArgs ra;
    ra.k_anchor = A.k_pool; ra.v_anchor = A.v_pool;
    ra.k_local = L.k_pool; ra.v_local = L.v_pool;
    ra.Wk = L.Wk_x; ra.Wv = L.Wv_x;
    ra.D = c->d.D; ra.m = c->d.m; ra.m_heads = c->d.m_heads;
    ra.part_tokens = c->d.part_tokens;
    ra.capacity_tokens = c->d.capacity;
    ScopedKernelTimer timer(c, s, ECHOKV_TIMED_RECON);
    if (!keys_whole) {
      ra.bk = L.bk_x;
      if (launch_recon_pair_store(a, ra, A.tc, L.tc, false, k_rows, c->d.capacity, c->d.D, c->sm_count, s) != cudaSuccess)
        return ECHOKV_ECUDA;
    }
    ra.bk = L.bv_x;
    if (launch_recon_pair_store(a, ra, A.tc, L.tc, true, v_rows, c->d.capacity, c->d.D, c->sm_count, s) != cudaSuccess)
      return ECHOKV_ECUDA;
    c->launches += keys_whole ? 1 : 2;
  }
  if (!windowed) {
    if (launch_prefill_attn(a, k_rows, v_rows, c->d.capacity, c->d.D, n_q, out, s) != cudaSuccess) return ECHOKV_ECUDA;
    c->launches += 1;
    return ECHOKV_OK;
  }
  // Section 4.1: every query's own sink and window at full precision.  The attention kernel covers what the query
  // sees as predicted (the sink left out, nothing closer than n_window positions); the band kernel adds the rest.
  float* lse = reinterpret_cast<float*>(static_cast<unsigned char*>(scratch) + 2 * rows_bytes);
  if (launch_prefill_attn(a, k_rows, v_rows, c->d.capacity, c->d.D, n_q, out, s, c->n_window, c->n_sink, lse) !=
      cudaSuccess)
    return ECHOKV_ECUDA;
  PrefillBand band;
  band.k_recent = k_recent; band.v_recent = v_recent;
  band.k_pool = L.k_pool; band.v_pool = L.v_pool;
  band.k_side = L.k_side; band.v_side = L.v_side;
  band.D = c->d.D; band.mk = c->d.mk; band.m = c->d.m; band.d_drop = c->d.d_drop;
  band.n_sink = c->n_sink; band.n_window = c->n_window;
  if (launch_prefill_band(a, band, n_q, out, lse, s) != cudaSuccess) return ECHOKV_ECUDA;
  c->launches += 2;
  return ECHOKV_OK;
}

int echokv_full_attention(echokv_ctx* c, int layer, const void* q, float* out,
                          const int32_t* dev_seq_slots, const int32_t* dev_seq_lens, int B,
                          void* stream) {
  const int rc = check_call(c, layer, q, out, dev_seq_lens, B);
  if (rc != ECHOKV_OK) return rc;
  const Layer& L = c->layers[layer];
  if (!L.anchor && c->d.d_drop != 0) return ECHOKV_ENOTANCHOR;
  return attend_stored_layer(c, L, q, out, dev_seq_slots, dev_seq_lens, B,
                             static_cast<cudaStream_t>(stream));
}

int echokv_decode_attention(echokv_ctx* c, int layer, const void* q, float* out,
                            const int32_t* dev_seq_slots, const int32_t* dev_seq_lens, int B,
                            void* stream) {
  const int rc = check_call(c, layer, q, out, dev_seq_lens, B);
  if (rc != ECHOKV_OK) return rc;
  const Layer& L = c->layers[layer];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (L.anchor || c->d.d_drop == 0)
    return attend_stored_layer(c, L, q, out, dev_seq_slots, dev_seq_lens, B, s);
  if (!L.Wv || (!L.Wk && !c->d.save_k)) return ECHOKV_ENOWEIGHTS;
  const Layer& A = c->layers[layer - layer % c->cfg.group_size];
  AttnArgs a = attn_args(c, q, dev_seq_slots, dev_seq_lens, B);
  const bool side = side_active(c, L);
  if (c->decode_mode == 1) {
    // absorbed predictors: every query head in one pass over [anchor dims ; retained dims]
    if (B > 256) return ECHOKV_EUNSUPPORTED;
    AbsorbArgs aa;
    aa.ws = c->ws_absorbed;
    aa.lay = c->alay;
    aa.Wk = L.Wk; aa.Wv = L.Wv; aa.bv = L.bv;
    aa.Wk_x = L.Wk_x; aa.bk_x = L.bk_x; aa.m_heads = c->d.m_heads;     // rotated keys: the explicit K pass
    aa.bk = c->rope.cs != nullptr ? L.bk : nullptr;
    aa.bk_shift = side && c->rope.cs == nullptr && !c->d.save_k ? L.bk : nullptr;
    aa.k_local = L.k_pool; aa.v_local = L.v_pool;
    aa.save_k = c->d.save_k;
    aa.D = c->d.D; aa.m = c->d.m;
    aa.capacity_tokens = c->d.capacity;
    aa.kernel_ms = nullptr;
    if (c->stored_capable && (c->d.save_k || c->d.m > 0)) {
      aa.k_stored = &L.stored_k;
      aa.k_stored_run = &L.stored_k_run;
    }
    if (side) {
      aa.n_sink = c->n_sink; aa.n_window = c->n_window;
      aa.k_side = L.k_side; aa.v_side = L.v_side;
    }
    cudaEvent_t ev[4];
    const bool timed = timed_pair(c, ECHOKV_TIMED_ABSORB_K, &ev[0], &ev[1]) &&
                       timed_pair(c, ECHOKV_TIMED_ABSORB_V, &ev[2], &ev[3]);
    if (launch_absorbed(a, aa, c->amaps, A.tc, L.tc, out, c->sm_count, s, timed ? ev : nullptr) != cudaSuccess)
      return ECHOKV_ECUDA;
    c->launches += (c->rope.cs != nullptr ? (c->d.save_k ? 5 : 5 + (c->d.m > 0 ? 1 : 0)) : 6) + (side ? 2 : 0);
    return ECHOKV_OK;
  }
  if (c->d.save_k) return ECHOKV_EUNSUPPORTED;   // explicit reconstruction predicts K as well: use the absorbed mode
  // whole retained heads; a head that m splits is predicted whole (its stored dims pass through the extended predictor)
  const int r = c->d.m_heads / c->cfg.head_dim;
  // retained heads: Eq. 7 on what is stored (Eq. 6 keeps them as they are)
  const int n_splits = stored_splits(c, B, r);
  const int32_t* item_tokens = nullptr;
  if (attend_stored_heads(c, a, L, c->d.m, r, n_splits, &item_tokens, s) != cudaSuccess) return ECHOKV_ECUDA;
  // dropped heads: predict (Eq. 3) and attend (Eq. 7) on chip
  ReconArgs ra;
  ra.k_anchor = A.k_pool; ra.v_anchor = A.v_pool;
  ra.k_local = L.k_pool; ra.v_local = L.v_pool;
  ra.Wk = L.Wk_x; ra.Wv = L.Wv_x;
  ra.bk = c->rope.cs != nullptr ? L.bk_x : nullptr;
  ra.D = c->d.D; ra.m = c->d.m; ra.m_heads = c->d.m_heads;
  ra.part_tokens = c->d.part_tokens;
  ra.capacity_tokens = c->d.capacity;
  ra.n_sink = side ? c->n_sink : 0;
  ra.n_window = side ? c->n_window : 0;
  cudaError_t e;
  const bool by_page_order = c->path == 5;
  if (by_page_order) {
    // both kernels are launched and the page order found in the block table says which of them runs
    if (launch_page_order(a, page_order_ptr(c), s) != cudaSuccess) return ECHOKV_ECUDA;
    ra.choose = page_order_ptr(c);
    c->launches += 2;
  }
  {
    ScopedKernelTimer timer(c, s, ECHOKV_TIMED_RECON);
    if (by_page_order) {
      ra.choose_value = 0;
      e = launch_recon_quad(a, ra, A.tc, L.tc, c->sm_count, s);
      if (e == cudaSuccess) {
        ra.choose_value = 1;
        e = launch_recon_tc(a, ra, A.tc, L.tc, c->sm_count, s);
      }
    } else if (c->path == 4) {
      e = launch_recon_quad(a, ra, A.tc, L.tc, c->sm_count, s);
    } else if (c->path == 3) {
      e = launch_recon_pair(a, ra, A.tc, L.tc, c->sm_count, s);
    } else if (c->path == 2) {
      e = launch_recon_tc(a, ra, A.tc, L.tc, c->sm_count, s);
    } else {
      e = launch_recon_simt(a, ra, s);
    }
  }
  if (e != cudaSuccess) return ECHOKV_ECUDA;
  const int recon_part_tokens = c->path == 2 ? kTcPartTokens : c->d.part_tokens;
  if (side) {
    // sink and recent-window tokens: Eq. 7 on their stored dims, one more partial per query head
    SidePool pool;
    pool.k_pool = L.k_pool; pool.v_pool = L.v_pool; pool.width = c->d.m; pool.part = -1;
    if (launch_attn_side(a, side_args(c, L), r, recon_part_tokens, s, pool, ra.choose, kTcPartTokens) != cudaSuccess)
      return ECHOKV_ECUDA;
    c->launches += 1;
  }
  // (a K bias is inside the scores already where the keys are rotated; otherwise it only matters against the
  // sink / window tokens, and the merge accounts for it)
  if (launch_merge(a, out, r, n_splits, item_tokens, kStoredMaxBatchPerLaunch, recon_part_tokens, L.bv_x, s,
                   side ? 1 : 0, side && c->rope.cs == nullptr ? L.bk_x : nullptr, ra.choose, kTcPartTokens) != cudaSuccess)
    return ECHOKV_ECUDA;
  c->launches += 2;
  return ECHOKV_OK;
}

int echokv_layer_step_host(echokv_ctx* c, int layer, const void* q_host, const void* k_new_host,
                           const void* v_new_host, float* out_host, const int32_t* seq_lens_host,
                           int B, int attend, void* stream) {
  if (!c || !k_new_host || !v_new_host || !seq_lens_host) return ECHOKV_EINVAL;
  if (attend && (!q_host || !out_host)) return ECHOKV_EINVAL;
  if (layer < 0 || layer >= c->cfg.n_layers || B < 1) return ECHOKV_EINVAL;
  if (B > c->cfg.max_batch) return ECHOKV_ECAPACITY;
  if (!c->table) return ECHOKV_ENOTABLE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const Derived& d = c->d;
  void* dq = c->ws + d.off_q;
  void* dk = c->ws + d.off_k;
  void* dv = c->ws + d.off_v;
  float* dout = reinterpret_cast<float*>(c->ws + d.off_out);
  int32_t* dlens = reinterpret_cast<int32_t*>(c->ws + d.off_lens);
  int32_t* dpos = reinterpret_cast<int32_t*>(c->ws + d.off_pos);
  const size_t q_bytes = (size_t)B * c->cfg.n_q_heads * c->cfg.head_dim * d.elem;
  const size_t kv_bytes = (size_t)B * d.D * d.elem;
  c->pos_scratch.resize(B);
  for (int b = 0; b < B; ++b) c->pos_scratch[b] = seq_lens_host[b] - 1;
  bool ok = true;
  ok &= cudaMemcpyAsync(dk, k_new_host, kv_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
  ok &= cudaMemcpyAsync(dv, v_new_host, kv_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
  ok &= cudaMemcpyAsync(dlens, seq_lens_host, (size_t)B * 4, cudaMemcpyHostToDevice, s) == cudaSuccess;
  ok &= cudaMemcpyAsync(dpos, c->pos_scratch.data(), (size_t)B * 4, cudaMemcpyHostToDevice, s) == cudaSuccess;
  if (attend) ok &= cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, s) == cudaSuccess;
  if (!ok) return ECHOKV_ECUDA;
  int rc = echokv_append_kv(c, layer, dk, dv, nullptr, dpos, B, stream);
  if (rc != ECHOKV_OK) return rc;
  if (attend) {
    rc = echokv_decode_attention(c, layer, dq, dout, nullptr, dlens, B, stream);
    if (rc != ECHOKV_OK) return rc;
    if (cudaMemcpyAsync(out_host, dout, (size_t)B * c->cfg.n_q_heads * c->cfg.head_dim * 4,
                        cudaMemcpyDeviceToHost, s) != cudaSuccess)
      return ECHOKV_ECUDA;
  }
  if (cudaStreamSynchronize(s) != cudaSuccess) return ECHOKV_ECUDA;
  return ECHOKV_OK;
}

int echokv_get_device_status(echokv_ctx* c, int32_t* host_out) {
  if (!c || !host_out) return ECHOKV_EINVAL;
  if (cudaDeviceSynchronize() != cudaSuccess) return ECHOKV_ECUDA;
  int32_t v = 0;
  if (cudaMemcpy(&v, status_ptr(c), 4, cudaMemcpyDeviceToHost) != cudaSuccess) return ECHOKV_ECUDA;
  if (v != 0 && cudaMemset(status_ptr(c), 0, 4) != cudaSuccess) return ECHOKV_ECUDA;
  *host_out = v;
  return ECHOKV_OK;
}

int echokv_set_kernel_timing(echokv_ctx* c, int enable) {
  if (!c) return ECHOKV_EINVAL;
  c->timing = enable != 0;
  return ECHOKV_OK;
}

int echokv_read_kernel_timing_by_kind(echokv_ctx* c, double* total_ms, int64_t* n_launches) {
  if (!c || !total_ms || !n_launches) return ECHOKV_EINVAL;
  if (cudaDeviceSynchronize() != cudaSuccess) return ECHOKV_ECUDA;
  for (int k = 0; k < ECHOKV_TIMED_KINDS; ++k) {
    total_ms[k] = 0.0;
    n_launches[k] = 0;
  }
  for (size_t i = 0; i < c->timed; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, c->events[i].first, c->events[i].second) != cudaSuccess) return ECHOKV_ECUDA;
    total_ms[c->event_kind[i]] += ms;
    n_launches[c->event_kind[i]] += 1;
  }
  c->timed = 0;
  return ECHOKV_OK;
}

int echokv_read_kernel_timing(echokv_ctx* c, double* total_ms, int64_t* n_launches) {
  if (!c || !total_ms || !n_launches) return ECHOKV_EINVAL;
  double ms[ECHOKV_TIMED_KINDS];
  int64_t n[ECHOKV_TIMED_KINDS];
  const int rc = echokv_read_kernel_timing_by_kind(c, ms, n);
  if (rc != ECHOKV_OK) return rc;
  *total_ms = 0.0;
  *n_launches = 0;
  for (int k = 0; k < ECHOKV_TIMED_KINDS; ++k) {
    *total_ms += ms[k];
    *n_launches += n[k];
  }
  return ECHOKV_OK;
}

int echokv_diag_page_order(echokv_ctx* c, int32_t* out) {
  if (!c || !out || c->path != 5) return ECHOKV_EINVAL;
  if (cudaDeviceSynchronize() != cudaSuccess) return ECHOKV_ECUDA;
  if (cudaMemcpy(out, page_order_ptr(c), sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return ECHOKV_ECUDA;
  return ECHOKV_OK;
}

int echokv_diag_bounded_wait(echokv_ctx* c, int64_t limit_cycles, int32_t* dev_left_by, void* stream) {
  if (!c || !dev_left_by || limit_cycles < 1 || limit_cycles > 2000000000ll) return ECHOKV_EINVAL;
  if (launch_bounded_wait_probe(status_ptr(c), limit_cycles, dev_left_by, static_cast<cudaStream_t>(stream)) !=
      cudaSuccess)
    return ECHOKV_ECUDA;
  c->launches += 1;
  return ECHOKV_OK;
}

int64_t echokv_launch_count(const echokv_ctx* c) { return c ? c->launches : 0; }

int echokv_decode_path(const echokv_ctx* c) { return c ? c->path : 0; }

const char* echokv_strerror(int status) {
  switch (status) {
    case ECHOKV_OK: return "ok";
    case ECHOKV_EINVAL: return "invalid argument";
    case ECHOKV_ENOTANCHOR: return "layer does not hold a full cache";
    case ECHOKV_ENOTCOMPRESSED: return "layer is an anchor layer and has no predictor";
    case ECHOKV_ECAPACITY: return "batch, workspace or length beyond the configured capacity";
    case ECHOKV_ENOWEIGHTS: return "predictor weights of the layer were not set";
    case ECHOKV_ECUDA: return "a CUDA call failed";
    case ECHOKV_ETIMEOUT: return "device: a bounded wait ran out";
    case ECHOKV_EBADPAGE: return "device: page id or sequence slot out of range";
    case ECHOKV_EUNSUPPORTED: return "shape not supported by the kernels";
    case ECHOKV_ENOTABLE: return "block table was not set";
    case ECHOKV_EBADLENGTH: return "device: sequence length below 1 or beyond capacity";
    case ECHOKV_ESCRATCH: return "problem does not fit the fixed scratch array of the no-alloc entry point";
    default: return "unknown status";
  }
}

}  // extern "C"
