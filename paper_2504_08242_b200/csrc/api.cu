// C-ABI layer: argument validation, context, dispatch.  See include/jupiter.h for the
// contract of every entry point.  All checks run on the host before anything is enqueued.
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/jupiter.h"
#include "host_checks.h"
#include "kernels.h"

struct jupiter_ctx {
  int device;
  int sm_count;
  void* workspace;
  size_t workspace_bytes;
  int* d_status;
  long long wait_limit;  // SM clocks a device-side wait may last
  int branch_kernel;     // jupiter_branch_kernel: which kernel the branch calls use
  uint64_t launches;
  char err[256];
};

namespace {

using jup::aligned16;
using jup::bf16;
using jup::CacheView;
using jup::check_cache;

jupiter_status cuda_fail(jupiter_ctx* ctx, cudaError_t e, const char* where) {
  if (ctx) std::snprintf(ctx->err, sizeof ctx->err, "%s: %s", where, cudaGetErrorString(e));
  return JUPITER_ERR_CUDA;
}

struct DeviceGuard {
  int prev;
  bool switched;
  explicit DeviceGuard(int dev) : prev(-1), switched(false) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

}  // namespace

extern "C" {

const char* jupiter_status_string(jupiter_status s) {
  switch (s) {
    case JUPITER_OK: return "ok";
    case JUPITER_ERR_INVALID_ARG: return "invalid argument";
    case JUPITER_ERR_OUT_OF_RANGE: return "position or length out of range";
    case JUPITER_ERR_UNSUPPORTED: return "unsupported shape or device";
    case JUPITER_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned";
    case JUPITER_ERR_WORKSPACE: return "context scratch too small";
    case JUPITER_ERR_CUDA: return "CUDA error";
    case JUPITER_ERR_TIMEOUT: return "bounded device wait expired";
  }
  return "unknown status";
}

jupiter_status jupiter_create(jupiter_ctx** out_ctx, int device, size_t workspace_bytes) {
  if (!out_ctx) return JUPITER_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  int count = 0;
  cudaError_t e = cudaGetDeviceCount(&count);
  if (e != cudaSuccess || device < 0 || device >= count) return e != cudaSuccess ? JUPITER_ERR_CUDA : JUPITER_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return JUPITER_ERR_CUDA;
  if (prop.major != 10) return JUPITER_ERR_UNSUPPORTED;  // kernels are built for sm_100a only
  jupiter_ctx* ctx = new (std::nothrow) jupiter_ctx();
  if (!ctx) return JUPITER_ERR_INVALID_ARG;
  std::memset(ctx, 0, sizeof *ctx);
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->workspace_bytes = workspace_bytes ? workspace_bytes : (size_t(64) << 20);
  ctx->wait_limit = 2000000000ll;
  DeviceGuard guard(device);
  e = cudaMalloc(&ctx->workspace, ctx->workspace_bytes);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ctx->d_status), 256);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 256);
  // the head of the scratch holds the branch kernel's completion counters, which must start at zero
  // (the kernel itself returns them to zero at the end of every call)
  if (e == cudaSuccess)
    e = cudaMemset(ctx->workspace, 0, ctx->workspace_bytes < 65536 ? ctx->workspace_bytes : size_t(65536));
  if (e != cudaSuccess) {
    if (ctx->workspace) cudaFree(ctx->workspace);
    if (ctx->d_status) cudaFree(ctx->d_status);
    delete ctx;
    return JUPITER_ERR_CUDA;
  }
  *out_ctx = ctx;
  return JUPITER_OK;
}

void jupiter_destroy(jupiter_ctx* ctx) {
  if (!ctx) return;
  DeviceGuard guard(ctx->device);
  cudaFree(ctx->workspace);
  cudaFree(ctx->d_status);
  delete ctx;
}

const char* jupiter_last_cuda_error(const jupiter_ctx* ctx) { return ctx ? ctx->err : ""; }

uint64_t jupiter_launch_count(const jupiter_ctx* ctx) { return ctx ? ctx->launches : 0; }

jupiter_status jupiter_poll_device_status(jupiter_ctx* ctx, void* stream) {
  if (!ctx) return JUPITER_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, ctx->d_status, sizeof word, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "poll");
  if (word != 0) {
    e = cudaMemsetAsync(ctx->d_status, 0, sizeof word, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "poll reset");
    return JUPITER_ERR_TIMEOUT;
  }
  return JUPITER_OK;
}

jupiter_status jupiter_select_branch_kernel(jupiter_ctx* ctx, jupiter_branch_kernel which) {
  if (!ctx || which < JUPITER_BRANCH_AUTO || which > JUPITER_BRANCH_TENSOR_CORE) return JUPITER_ERR_INVALID_ARG;
  ctx->branch_kernel = which;
  return JUPITER_OK;
}

jupiter_status jupiter_wait_probe(jupiter_ctx* ctx, int64_t limit_cycles, void* stream) {
  if (!ctx || limit_cycles <= 0 || limit_cycles > 2000000000ll) return JUPITER_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaError_t e = jup::launch_wait_probe(ctx->d_status, limit_cycles, static_cast<cudaStream_t>(stream), li);
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "wait_probe");
}

jupiter_status jupiter_read_probe(jupiter_ctx* ctx, const void* src, size_t bytes, uint32_t* out, void* stream) {
  if (!ctx || !src || !out) return JUPITER_ERR_INVALID_ARG;
  if (!aligned16(src) || (bytes % 16) != 0) return JUPITER_ERR_ALIGNMENT;
  if (bytes == 0) return JUPITER_OK;
  DeviceGuard guard(ctx->device);
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaError_t e = jup::launch_read_probe(src, bytes, out, static_cast<cudaStream_t>(stream), li);
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "read_probe");
}

jupiter_status jupiter_kv_append(jupiter_ctx* ctx, const jupiter_kv_cache* cache, const void* k_new,
                                 const void* v_new, int32_t n_rows, int32_t pos, const int32_t* d_pos,
                                 void* stream) {
  if (!ctx || !k_new || !v_new) return JUPITER_ERR_INVALID_ARG;
  CacheView c;
  jupiter_status s = check_cache(cache, &c);
  if (s != JUPITER_OK) return s;
  if (n_rows < 0) return JUPITER_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return JUPITER_ERR_ALIGNMENT;
  if (d_pos) {
    if (n_rows > c.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  } else {
    if (pos < 0 || static_cast<int64_t>(pos) + n_rows > c.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  }
  if (n_rows == 0) return JUPITER_OK;
  DeviceGuard guard(ctx->device);
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaError_t e = jup::launch_kv_append(c, static_cast<const bf16*>(k_new), static_cast<const bf16*>(v_new), n_rows,
                                        pos, d_pos, static_cast<cudaStream_t>(stream), li);
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "kv_append");
}

jupiter_status jupiter_kv_compact(jupiter_ctx* ctx, const jupiter_kv_cache* cache, int32_t q_len,
                                  const int32_t* d_pos, const int32_t* d_accept, const int32_t* d_n_accept,
                                  void* stream) {
  if (!ctx || !d_pos || !d_accept || !d_n_accept) return JUPITER_ERR_INVALID_ARG;
  CacheView c;
  jupiter_status s = check_cache(cache, &c);
  if (s != JUPITER_OK) return s;
  if (q_len <= 0) return JUPITER_ERR_INVALID_ARG;
  if (q_len > 16) return JUPITER_ERR_UNSUPPORTED;
  if (q_len > c.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  if (static_cast<int64_t>(c.batch) * c.kv_heads > 0x7fffffff) return JUPITER_ERR_UNSUPPORTED;
  DeviceGuard guard(ctx->device);
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaError_t e = jup::launch_kv_compact(c, q_len, d_pos, d_accept, d_n_accept, static_cast<cudaStream_t>(stream), li);
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "kv_compact");
}

jupiter_status jupiter_chunk_prefill_attn(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* cache,
                                          int32_t q_heads, int32_t q_len, int32_t pos, float scale, float* out,
                                          float* lse, void* stream) {
  if (!ctx || !q || !out) return JUPITER_ERR_INVALID_ARG;
  CacheView c;
  jupiter_status s = check_cache(cache, &c);
  if (s != JUPITER_OK) return s;
  if (q_heads <= 0 || q_len <= 0 || q_heads % c.kv_heads != 0) return JUPITER_ERR_INVALID_ARG;
  if (!jup::scale_ok(scale)) return JUPITER_ERR_INVALID_ARG;
  if (pos < 0 || static_cast<int64_t>(pos) + q_len > c.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  if (!aligned16(q) || !aligned16(out)) return JUPITER_ERR_ALIGNMENT;
  DeviceGuard guard(ctx->device);
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaError_t e;
  if (jup::prefill_tc_supported(c, scale))
    e = jup::launch_prefill_tc(static_cast<const bf16*>(q), c, nullptr, 0, q_heads, q_len, pos, scale, out, lse,
                               ctx->d_status, ctx->workspace, ctx->workspace_bytes, static_cast<cudaStream_t>(stream), li);
  else  // head_dim 64, or a non-positive scale: the general mma.sync kernel
    e = jup::launch_prefill_mma(static_cast<const bf16*>(q), c, q_heads, q_len, pos, scale, out, lse,
                                static_cast<cudaStream_t>(stream), li);
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "chunk_prefill_attn");
}

jupiter_status jupiter_chunk_prefill_append_attn(jupiter_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                                 const jupiter_kv_cache* cache, int32_t q_heads, int32_t q_len,
                                                 int32_t pos, float scale, float* out, float* lse, void* stream) {
  if (!ctx || !q || !k_new || !v_new || !out) return JUPITER_ERR_INVALID_ARG;
  CacheView c;
  jupiter_status s = check_cache(cache, &c);
  if (s != JUPITER_OK) return s;
  if (q_heads <= 0 || q_len <= 0 || q_heads % c.kv_heads != 0) return JUPITER_ERR_INVALID_ARG;
  if (!jup::scale_ok(scale)) return JUPITER_ERR_INVALID_ARG;
  if (pos < 0 || static_cast<int64_t>(pos) + q_len > c.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  if (!aligned16(q) || !aligned16(out) || !aligned16(k_new) || !aligned16(v_new)) return JUPITER_ERR_ALIGNMENT;
  DeviceGuard guard(ctx->device);
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (jup::prefill_tc_supported(c, scale)) {
    e = jup::launch_prefill_tc_fused(static_cast<const bf16*>(q), c, static_cast<const bf16*>(k_new),
                                     static_cast<const bf16*>(v_new), q_heads, q_len, pos, scale, out, lse,
                                     ctx->d_status, ctx->workspace, ctx->workspace_bytes, st, li);
  } else {  // head_dim 64, or a non-positive scale: the append kernel, then the general mma.sync kernel
    e = jup::launch_kv_append(c, static_cast<const bf16*>(k_new), static_cast<const bf16*>(v_new), q_len, pos, nullptr,
                              st, li);
    if (e == cudaSuccess)
      e = jup::launch_prefill_mma(static_cast<const bf16*>(q), c, q_heads, q_len, pos, scale, out, lse, st, li);
  }
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "chunk_prefill_append_attn");
}

jupiter_status jupiter_branch_prefill_attn(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* prefix,
                                          int32_t prefix_len, const jupiter_kv_cache* cache, int32_t q_heads,
                                          int32_t q_len, int32_t pos, float scale, float* out, float* lse,
                                          void* stream) {
  if (!ctx || !q || !out) return JUPITER_ERR_INVALID_ARG;
  CacheView c;
  jupiter_status s = check_cache(cache, &c);
  if (s != JUPITER_OK) return s;
  CacheView pfx = c;
  if (prefix_len < 0) return JUPITER_ERR_INVALID_ARG;
  if (prefix_len > 0) {
    s = check_cache(prefix, &pfx);
    if (s != JUPITER_OK) return s;
    if (pfx.batch != 1 || pfx.kv_heads != c.kv_heads || pfx.head_dim != c.head_dim) return JUPITER_ERR_INVALID_ARG;
    if (prefix_len > pfx.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  }
  if (q_heads <= 0 || q_len <= 0 || q_heads % c.kv_heads != 0) return JUPITER_ERR_INVALID_ARG;
  if (!jup::scale_ok(scale)) return JUPITER_ERR_INVALID_ARG;
  if (pos < 0 || static_cast<int64_t>(pos) + q_len > c.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  if (!aligned16(q) || !aligned16(out)) return JUPITER_ERR_ALIGNMENT;
  if (!jup::prefill_tc_supported(c, scale)) return JUPITER_ERR_UNSUPPORTED;  // head_dim 128 and scale > 0 only
  DeviceGuard guard(ctx->device);
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaError_t e = jup::launch_prefill_tc(static_cast<const bf16*>(q), c, prefix_len > 0 ? &pfx : nullptr, prefix_len,
                                         q_heads, q_len, pos, scale, out, lse, ctx->d_status, ctx->workspace,
                                         ctx->workspace_bytes, static_cast<cudaStream_t>(stream), li);
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "branch_prefill_attn");
}

static jupiter_status branch_attn_impl(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* prefix,
                                       int32_t prefix_len, const jupiter_kv_cache* suffix,
                                       const int32_t* d_suffix_len, const uint32_t* d_tree_mask,
                                       int32_t max_suffix_len, int32_t n_branches, int32_t q_heads, int32_t q_len,
                                       float scale, float* out, float* lse, void* stream, const void* k_new = nullptr,
                                       const void* v_new = nullptr) {
  if (!ctx || !q || !out || !d_suffix_len) return JUPITER_ERR_INVALID_ARG;
  if (!aligned16(k_new) || !aligned16(v_new)) return JUPITER_ERR_ALIGNMENT;
  CacheView sfx;
  jupiter_status s = check_cache(suffix, &sfx);
  if (s != JUPITER_OK) return s;
  CacheView pfx = sfx;
  if (prefix_len < 0) return JUPITER_ERR_INVALID_ARG;
  if (prefix_len > 0) {
    s = check_cache(prefix, &pfx);
    if (s != JUPITER_OK) return s;
    if (pfx.batch != 1 || pfx.kv_heads != sfx.kv_heads || pfx.head_dim != sfx.head_dim) return JUPITER_ERR_INVALID_ARG;
    if (prefix_len > pfx.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  }
  if (n_branches <= 0 || n_branches != sfx.batch) return JUPITER_ERR_INVALID_ARG;
  if (q_heads <= 0 || q_heads % sfx.kv_heads != 0 || q_len <= 0) return JUPITER_ERR_INVALID_ARG;
  if (q_len > 16) return JUPITER_ERR_UNSUPPORTED;
  if (!jup::scale_ok(scale)) return JUPITER_ERR_INVALID_ARG;
  if (max_suffix_len < q_len || max_suffix_len > sfx.capacity) return JUPITER_ERR_OUT_OF_RANGE;
  if (!aligned16(q) || !aligned16(out)) return JUPITER_ERR_ALIGNMENT;
  // which kernel: few stacked rows per kv head stream through clusters (no scratch); many rows with head_dim 128 go
  // to the tensor-core kernel (which adapts to the scratch it is given); the rest to the split-KV kernel, the only one that can find the
  // scratch too small
  DeviceGuard guard(ctx->device);
  const bool tc_ok = jup::branch_tc_supported(sfx, prefix_len, max_suffix_len, n_branches, q_heads, q_len, scale,
                                              ctx->sm_count);
  bool use_stream, use_tc;
  switch (ctx->branch_kernel) {
    case JUPITER_BRANCH_STREAM: use_stream = true, use_tc = false; break;
    case JUPITER_BRANCH_SPLIT_KV: use_stream = use_tc = false; break;
    case JUPITER_BRANCH_TENSOR_CORE:
      if (!tc_ok) return JUPITER_ERR_UNSUPPORTED;
      use_stream = false, use_tc = true;
      break;
    default:
      use_stream = jup::branch_stream_preferred(n_branches, q_heads, sfx.kv_heads, q_len, ctx->sm_count);
      use_tc = !use_stream && tc_ok;
  }
  if (!use_stream && !use_tc &&
      jup::branch_workspace_bytes(prefix_len, max_suffix_len, n_branches, q_heads, sfx.kv_heads, q_len, sfx.head_dim,
                                  ctx->sm_count) > ctx->workspace_bytes)
    return JUPITER_ERR_WORKSPACE;
  jup::LaunchInfo li{ctx->sm_count, 0};
  cudaError_t e;
  if (use_stream)
    e = jup::launch_branch_stream(static_cast<const bf16*>(q), pfx, prefix_len, sfx, d_suffix_len, d_tree_mask,
                                  max_suffix_len, n_branches, q_heads, q_len, scale, out, lse,
                                  static_cast<cudaStream_t>(stream), li, static_cast<const bf16*>(k_new),
                                  static_cast<const bf16*>(v_new));
  else if (use_tc)
    e = jup::launch_branch_tc(static_cast<const bf16*>(q), pfx, prefix_len, sfx, d_suffix_len, d_tree_mask,
                              max_suffix_len, n_branches, q_heads, q_len, scale, out, lse, ctx->d_status,
                              ctx->wait_limit, ctx->workspace, ctx->workspace_bytes, static_cast<cudaStream_t>(stream),
                              li, static_cast<const bf16*>(k_new), static_cast<const bf16*>(v_new));
  else
    e = jup::launch_branch(static_cast<const bf16*>(q), pfx, prefix_len, sfx, d_suffix_len, d_tree_mask,
                           max_suffix_len, n_branches, q_heads, q_len, scale, out, lse, ctx->workspace,
                           static_cast<cudaStream_t>(stream), li, static_cast<const bf16*>(k_new),
                           static_cast<const bf16*>(v_new));
  ctx->launches += li.launches;
  return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "branch_attn");
}

jupiter_status jupiter_branch_append_attn_layers(jupiter_ctx* ctx, const jupiter_branch_layer* layers,
                                                 int32_t n_layers, int32_t prefix_len, const int32_t* d_suffix_len,
                                                 int32_t max_suffix_len, int32_t n_branches, int32_t q_heads,
                                                 int32_t q_len, float scale, void* stream) {
  if (!ctx || !layers || n_layers <= 0 || !d_suffix_len) return JUPITER_ERR_INVALID_ARG;
  if (prefix_len < 0 || n_branches <= 0 || q_heads <= 0 || q_len <= 0) return JUPITER_ERR_INVALID_ARG;
  if (q_len > 16) return JUPITER_ERR_UNSUPPORTED;
  if (!jup::scale_ok(scale)) return JUPITER_ERR_INVALID_ARG;
  // every layer is checked before anything is enqueued
  CacheView sfx0, pfx0;
  std::vector<jup::BranchLayerTensors> t(static_cast<size_t>(n_layers));
  for (int l = 0; l < n_layers; ++l) {
    const jupiter_branch_layer& L = layers[l];
    if (!L.q || !L.k_new || !L.v_new || !L.out) return JUPITER_ERR_INVALID_ARG;
    if (!aligned16(L.q) || !aligned16(L.k_new) || !aligned16(L.v_new) || !aligned16(L.out)) return JUPITER_ERR_ALIGNMENT;
    CacheView sfx;
    jupiter_status s = check_cache(L.suffix, &sfx);
    if (s != JUPITER_OK) return s;
    CacheView pfx = sfx;
    if (prefix_len > 0) {
      s = check_cache(L.prefix, &pfx);
      if (s != JUPITER_OK) return s;
      if (pfx.batch != 1 || pfx.kv_heads != sfx.kv_heads || pfx.head_dim != sfx.head_dim) return JUPITER_ERR_INVALID_ARG;
      if (prefix_len > pfx.capacity) return JUPITER_ERR_OUT_OF_RANGE;
    }
    if (n_branches != sfx.batch || q_heads % sfx.kv_heads != 0) return JUPITER_ERR_INVALID_ARG;
    if (max_suffix_len < q_len || max_suffix_len > sfx.capacity) return JUPITER_ERR_OUT_OF_RANGE;
    if (l == 0) {
      sfx0 = sfx;
      pfx0 = pfx;
    } else {
      auto same = [](const CacheView& a, const CacheView& b) {
        return a.batch == b.batch && a.kv_heads == b.kv_heads && a.capacity == b.capacity && a.head_dim == b.head_dim &&
               a.sb == b.sb && a.sh == b.sh && a.sr == b.sr;
      };
      if (!same(sfx, sfx0) || (prefix_len > 0 && !same(pfx, pfx0))) return JUPITER_ERR_INVALID_ARG;
    }
    t[l] = jup::BranchLayerTensors{static_cast<const bf16*>(L.q), static_cast<const bf16*>(L.k_new),
                                   static_cast<const bf16*>(L.v_new), pfx.k, pfx.v, sfx.k, sfx.v, L.out, L.lse};
  }
  if (ctx->branch_kernel == JUPITER_BRANCH_AUTO &&
      jup::branch_stream_preferred(n_branches, q_heads, sfx0.kv_heads, q_len, ctx->sm_count)) {
    DeviceGuard guard(ctx->device);
    jup::LaunchInfo li{ctx->sm_count, 0};
    cudaError_t e = jup::launch_branch_stream_layers(t.data(), n_layers, pfx0, prefix_len, sfx0, d_suffix_len,
                                                     max_suffix_len, n_branches, q_heads, q_len, scale,
                                                     static_cast<cudaStream_t>(stream), li);
    ctx->launches += li.launches;
    return e == cudaSuccess ? JUPITER_OK : cuda_fail(ctx, e, "branch_append_attn_layers");
  }
  // the other kernels take the layers one by one (arguments are known to be valid; a layer can still find the
  // context's scratch too small, before its own launch)
  for (int l = 0; l < n_layers; ++l) {
    const jupiter_branch_layer& L = layers[l];
    jupiter_status s = branch_attn_impl(ctx, L.q, L.prefix, prefix_len, L.suffix, d_suffix_len, nullptr, max_suffix_len,
                                        n_branches, q_heads, q_len, scale, L.out, L.lse, stream, L.k_new, L.v_new);
    if (s != JUPITER_OK) return s;
  }
  return JUPITER_OK;
}

jupiter_status jupiter_branch_append_attn(jupiter_ctx* ctx, const void* q, const void* k_new, const void* v_new,
                                          const jupiter_kv_cache* prefix, int32_t prefix_len,
                                          const jupiter_kv_cache* suffix, const int32_t* d_suffix_len,
                                          int32_t max_suffix_len, int32_t n_branches, int32_t q_heads, int32_t q_len,
                                          float scale, float* out, float* lse, void* stream) {
  if (!k_new || !v_new) return JUPITER_ERR_INVALID_ARG;
  return branch_attn_impl(ctx, q, prefix, prefix_len, suffix, d_suffix_len, nullptr, max_suffix_len, n_branches,
                          q_heads, q_len, scale, out, lse, stream, k_new, v_new);
}

jupiter_status jupiter_branch_attn(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* prefix,
                                   int32_t prefix_len, const jupiter_kv_cache* suffix, const int32_t* d_suffix_len,
                                   int32_t max_suffix_len, int32_t n_branches, int32_t q_heads, int32_t q_len,
                                   float scale, float* out, float* lse, void* stream) {
  return branch_attn_impl(ctx, q, prefix, prefix_len, suffix, d_suffix_len, nullptr, max_suffix_len, n_branches,
                          q_heads, q_len, scale, out, lse, stream);
}

jupiter_status jupiter_branch_attn_tree(jupiter_ctx* ctx, const void* q, const jupiter_kv_cache* prefix,
                                        int32_t prefix_len, const jupiter_kv_cache* suffix,
                                        const int32_t* d_suffix_len, const uint32_t* d_tree_mask,
                                        int32_t max_suffix_len, int32_t n_branches, int32_t q_heads, int32_t q_len,
                                        float scale, float* out, float* lse, void* stream) {
  if (!d_tree_mask) return JUPITER_ERR_INVALID_ARG;
  return branch_attn_impl(ctx, q, prefix, prefix_len, suffix, d_suffix_len, d_tree_mask, max_suffix_len, n_branches,
                          q_heads, q_len, scale, out, lse, stream);
}

}  // extern "C"
