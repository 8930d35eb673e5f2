// echokv_full_attention_noalloc: full-cache attention for callers that cannot allocate.
//
// The regular entry points keep their split-K partial results in a workspace that the caller
// allocates.  Some callers have no allocator to ask: code that runs inside another framework's
// execution callback where device allocation is forbidden, or a host thread that is only handed
// raw pointers to an arena sized long ago.  For them this file keeps the scratch in a fixed
// device array that is part of the library image.  The paper has no counterpart to this.
#include <cmath>
#include <mutex>

#include "kernels.h"

using namespace echokv;

namespace {

constexpr size_t kScratchBytes = 8u << 20;   // 8 MiB, held by every device that loads the library
constexpr size_t kStatusBytes = 256;
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is
// not a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_scratch on this device
  int sm_count = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Once per device, with that device current.
int setup_device(int device, DeviceSetup** out) {
  if (device < 0 || device >= kMaxDevices) return ECHOKV_EINVAL;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& s = g_setup[device];
  if (!s.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || ptr == nullptr) return ECHOKV_ECUDA;
    if (cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
      return ECHOKV_ECUDA;
    s.scratch = static_cast<unsigned char*>(ptr);
    s.ready = true;
  }
  *out = &s;
  return ECHOKV_OK;
}

size_t partial_bytes(int B, int n_q_heads, int head_dim, int n_splits) {
  const size_t n = (size_t)B * n_q_heads * n_splits;
  const size_t ml = (n * sizeof(float2) + 255) / 256 * 256;
  return kStatusBytes + ml + n * head_dim * sizeof(float);
}

}  // namespace

extern "C" int echokv_full_attention_noalloc(const echokv_config* cfg, const void* k_pool,
                                             const void* v_pool, const int32_t* dev_block_table,
                                             const void* q, float* out, const int32_t* dev_seq_slots,
                                             const int32_t* dev_seq_lens, int B,
                                             int32_t* dev_status_out, void* stream) {
  if (!cfg || !k_pool || !v_pool || !dev_block_table || !q || !out || !dev_seq_lens) return ECHOKV_EINVAL;
  if (cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->n_q_heads % cfg->n_kv_heads != 0) return ECHOKV_EINVAL;
  if (cfg->max_batch < 1 || cfg->max_pages_per_seq < 1 || cfg->n_pages < 1 || B < 1) return ECHOKV_EINVAL;
  if (cfg->dtype != ECHOKV_BF16 && cfg->dtype != ECHOKV_FP32) return ECHOKV_EINVAL;
  if (!(cfg->softmax_scale >= 0.f) || !std::isfinite(cfg->softmax_scale)) return ECHOKV_EINVAL;
  // a capacity beyond 2^30 tokens would overflow the kernels' int arithmetic on lengths
  if ((long long)cfg->max_pages_per_seq * cfg->page_tokens > (1ll << 30)) return ECHOKV_EINVAL;
  // the kernel reads the pools and the queries with 16-byte loads: a pointer aligned to less would fault on
  // the device instead of returning a status
  if ((reinterpret_cast<uintptr_t>(k_pool) | reinterpret_cast<uintptr_t>(v_pool) | reinterpret_cast<uintptr_t>(q) |
       reinterpret_cast<uintptr_t>(out)) % 16 != 0)
    return ECHOKV_EINVAL;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return ECHOKV_EUNSUPPORTED;
  if (cfg->page_tokens != 16 && cfg->page_tokens != 32 && cfg->page_tokens != 64 && cfg->page_tokens != 128)
    return ECHOKV_EUNSUPPORTED;
  const int g = cfg->n_q_heads / cfg->n_kv_heads;
  if (g != 1 && g != 2 && g != 4 && g != 8) return ECHOKV_EUNSUPPORTED;
  if (B > cfg->max_batch) return ECHOKV_ECAPACITY;
  // even a single partial per (sequence, head) must fit the fixed scratch
  if (partial_bytes(B, cfg->n_q_heads, cfg->head_dim, 1) > kScratchBytes) return ECHOKV_ESCRATCH;

  if (cudaSetDevice(cfg->device) != cudaSuccess) return ECHOKV_ECUDA;
  DeviceSetup* dev = nullptr;
  const int rc = setup_device(cfg->device, &dev);
  if (rc != ECHOKV_OK) return rc;

  int n_splits = (4 * dev->sm_count + B * cfg->n_kv_heads - 1) / (B * cfg->n_kv_heads);
  if (n_splits > cfg->max_pages_per_seq) n_splits = cfg->max_pages_per_seq;
  if (n_splits < 1) n_splits = 1;
  while (n_splits > 1 && partial_bytes(B, cfg->n_q_heads, cfg->head_dim, n_splits) > kScratchBytes) --n_splits;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  unsigned char* base = dev->scratch;   // the address cudaGetSymbolAddress returned
  int32_t* status = reinterpret_cast<int32_t*>(base);
  // the scratch keeps what the previous call left: the status word is the only part read before
  // it is written, so it is the only part cleared
  if (cudaMemsetAsync(status, 0, sizeof(int32_t), s) != cudaSuccess) return ECHOKV_ECUDA;

  const size_t n = (size_t)B * cfg->n_q_heads * n_splits;
  AttnArgs a;
  a.dtype = cfg->dtype;
  a.n_q_heads = cfg->n_q_heads;
  a.n_kv_heads = cfg->n_kv_heads;
  a.head_dim = cfg->head_dim;
  a.batch = B;
  const float scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
  a.scale_log2e = scale * kLog2e;
  a.q = q;
  a.slots = dev_seq_slots;
  a.lens = dev_seq_lens;
  a.geom.table = dev_block_table;
  a.geom.max_batch = cfg->max_batch;
  a.geom.max_pages_per_seq = cfg->max_pages_per_seq;
  a.geom.page_tokens = cfg->page_tokens;
  a.geom.n_pages = cfg->n_pages;
  a.parts.ml = reinterpret_cast<float2*>(base + kStatusBytes);
  a.parts.o = reinterpret_cast<float*>(base + kStatusBytes + (n * sizeof(float2) + 255) / 256 * 256);
  a.parts.max_parts = n_splits;
  a.status = status;
  const int D = cfg->n_kv_heads * cfg->head_dim;
  if (launch_attn_stored(a, k_pool, v_pool, D, cfg->n_kv_heads, n_splits, s) != cudaSuccess) return ECHOKV_ECUDA;
  if (launch_merge(a, out, cfg->n_kv_heads, n_splits, nullptr, 1, /*part_tokens=*/1, nullptr, s) != cudaSuccess)
    return ECHOKV_ECUDA;
  if (dev_status_out &&
      cudaMemcpyAsync(dev_status_out, status, sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return ECHOKV_ECUDA;
  return ECHOKV_OK;
}

extern "C" uint64_t echokv_noalloc_scratch_bytes(void) { return kScratchBytes; }
