// jupiter_branch_attn_noalloc: branch attention for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need
// attention: code running inside a memory pool that owns the whole device, a plugin
// whose host framework forbids allocator calls on its worker threads, or a serving
// loop that has promised a fixed memory footprint after start-up.  For them the split-KV
// scratch of jupiter_branch_attn lives in a fixed array inside the library image instead
// of a context's cudaMalloc'd workspace.  No jupiter_ctx is involved at all.
#include <mutex>

#include "../../include/jupiter.h"
#include "host_checks.h"
#include "kernels.h"

// The scratch itself: part of the loaded module, so every GPU that loads the library
// holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[JUPITER_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
struct PerDevice {
  bool ready;
  void* scratch;  // device address of g_noalloc_scratch on that device
  int sm_count;
};
PerDevice g_dev[kMaxDevices];
std::mutex g_mu;

// One-time set-up for the current device.  In host code the name g_noalloc_scratch is only
// a host-side handle of the symbol, not something a kernel can dereference; the address
// the GPU sees has to be asked for, with the device in question current.
jupiter_status device_setup(int dev, PerDevice** out) {
  if (dev < 0 || dev >= kMaxDevices) return JUPITER_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  PerDevice& d = g_dev[dev];
  if (!d.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return JUPITER_ERR_CUDA;
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return JUPITER_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return JUPITER_ERR_CUDA;
    if (major != 10) return JUPITER_ERR_UNSUPPORTED;
    d.scratch = ptr;
    d.sm_count = sms;
    d.ready = true;
  }
  *out = &d;
  return JUPITER_OK;
}

}  // namespace

extern "C" jupiter_status jupiter_branch_attn_noalloc(const void* q, const jupiter_kv_cache* prefix,
                                                      int32_t prefix_len, const jupiter_kv_cache* suffix,
                                                      const int32_t* d_suffix_len, int32_t max_suffix_len,
                                                      int32_t n_branches, int32_t q_heads, int32_t q_len,
                                                      float scale, float* out, float* lse, void* stream) {
  if (!q || !out || !d_suffix_len) return JUPITER_ERR_INVALID_ARG;
  jup::CacheView sfx;
  jupiter_status s = jup::check_cache(suffix, &sfx);
  if (s != JUPITER_OK) return s;
  jup::CacheView pfx = sfx;
  if (prefix_len < 0) return JUPITER_ERR_INVALID_ARG;
  if (prefix_len > 0) {
    s = jup::check_cache(prefix, &pfx);
    if (s != JUPITER_OK) return s;
    if (pfx.batch != 1 || pfx.kv_heads != sfx.kv_heads || pfx.head_dim != sfx.head_dim) return JUPITER_ERR_INVALID_ARG;
    if (prefix_len > pfx.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  }
  if (n_branches <= 0 || n_branches != sfx.batch) return JUPITER_ERR_INVALID_ARG;
  if (q_heads <= 0 || q_heads % sfx.kv_heads != 0 || q_len <= 0) return JUPITER_ERR_INVALID_ARG;
  if (q_len > 16) return JUPITER_ERR_UNSUPPORTED;
  if (!jup::scale_ok(scale)) return JUPITER_ERR_INVALID_ARG;
  if (max_suffix_len < q_len || max_suffix_len > sfx.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  if (!jup::aligned16(q) || !jup::aligned16(out)) return JUPITER_ERR_ALIGNMENT;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return JUPITER_ERR_CUDA;
  PerDevice* d = nullptr;
  s = device_setup(dev, &d);
  if (s != JUPITER_OK) return s;

  const size_t need = jup::branch_workspace_bytes(prefix_len, max_suffix_len, n_branches, q_heads, sfx.kv_heads, q_len,
                                                  sfx.head_dim, d->sm_count);
  if (need > static_cast<size_t>(JUPITER_NOALLOC_SCRATCH_BYTES)) return JUPITER_ERR_WORKSPACE;

  // What must be zero when a call starts are the completion counters at the head of the array.  They
  // are zero when the module is loaded, and the kernel puts each one back to zero once the last
  // contributor of its group has reported, so no clearing pass is needed between calls.  The partial
  // results behind them are fully rewritten before they are read.
  jup::LaunchInfo li{d->sm_count, 0};
  cudaError_t e = jup::launch_branch(static_cast<const jup::bf16*>(q), pfx, prefix_len, sfx, d_suffix_len, nullptr,
                                     max_suffix_len, n_branches, q_heads, q_len, scale, out, lse, d->scratch,
                                     static_cast<cudaStream_t>(stream), li);
  return e == cudaSuccess ? JUPITER_OK : JUPITER_ERR_CUDA;
}
