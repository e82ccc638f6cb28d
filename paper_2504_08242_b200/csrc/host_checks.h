// Host-side argument checks shared by the C-ABI entry points, and a per-device "done once" flag for the
// launchers (function attributes are per device).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cmath>

#include "../../include/jupiter.h"
#include "kernels.h"

namespace jup {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The softmax scale must be a finite number (NaN and +-inf are refused before anything is enqueued).
inline bool scale_ok(float scale) { return std::isfinite(scale); }

// Validates a cache descriptor and turns it into a CacheView.  A dimension with more than one entry needs
// a non-zero stride: a broadcast cache (stride 0) is refused rather than silently read at a wrong address by
// the tensor-map kernels, which cannot encode it.
inline jupiter_status check_cache(const jupiter_kv_cache* c, CacheView* out) {
  if (!c || !c->k || !c->v) return JUPITER_ERR_INVALID_ARG;
  if (c->batch <= 0 || c->kv_heads <= 0 || c->capacity <= 0) return JUPITER_ERR_INVALID_ARG;
  if (c->head_dim != 64 && c->head_dim != 128) return JUPITER_ERR_UNSUPPORTED;
  if (c->stride_row < c->head_dim || c->stride_head < 0 || c->stride_batch < 0) return JUPITER_ERR_INVALID_ARG;
  if ((c->kv_heads > 1 && c->stride_head == 0) || (c->batch > 1 && c->stride_batch == 0)) return JUPITER_ERR_INVALID_ARG;
  if (!aligned16(c->k) || !aligned16(c->v)) return JUPITER_ERR_ALIGNMENT;
  if ((c->stride_row % 8) || (c->stride_head % 8) || (c->stride_batch % 8)) return JUPITER_ERR_ALIGNMENT;
  out->k = static_cast<const bf16*>(c->k);
  out->v = static_cast<const bf16*>(c->v);
  out->batch = c->batch;
  out->kv_heads = c->kv_heads;
  out->capacity = c->capacity;
  out->head_dim = c->head_dim;
  out->sb = c->stride_batch;
  out->sh = c->stride_head;
  out->sr = c->stride_row;
  return JUPITER_OK;
}

// One flag per CUDA device: `if (!flag.done()) { ...set attributes...; flag.set(); }` runs the body at least once on
// every device a launcher is used on (a second thread may repeat it, which is harmless for attribute calls).
class PerDeviceOnce {
 public:
  bool done() const {
    const int d = index();
    return d >= 0 && flags_[d].load(std::memory_order_acquire);
  }
  void set() {
    const int d = index();
    if (d >= 0) flags_[d].store(true, std::memory_order_release);
  }

 private:
  static constexpr int kMax = 64;
  static int index() {
    int d = -1;
    return (cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < kMax) ? d : -1;
  }
  std::atomic<bool> flags_[kMax] = {};
};

}  // namespace jup
