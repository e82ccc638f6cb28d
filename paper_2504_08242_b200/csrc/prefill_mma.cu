// Chunked-prefill attention on mma.sync (paper Sec. IV-A, Fig. 5(b)): the chunk's
// rows at positions pos..pos+n-1 attend to cache rows 0..pos+i.  General-shape
// path: any head_dim in {64,128}, any pos / q_len.  One CTA = 64 chunk rows of
// one (sequence, query head); heaviest row tiles are scheduled first.
#include "attn_mma.cuh"
#include "host_checks.h"
#include "kernels.h"

namespace jup {

struct PrefillParams {
  const bf16* q;
  CacheView c;
  int q_heads, group, q_len, pos, tiles;
  float scale_log2;
  float* out;
  float* lse;
};

template <int D>
struct PrefillItem {
  const bf16* k;
  const bf16* v;
  int64_t row_stride;
  int kv_begin, kv_end;
  bool partial;
  // row mapping
  const bf16* q;
  float* out;
  float* lse;
  int row0, q_len, pos;
  int64_t q_tok_stride;  // elements between consecutive chunk rows of this head
  __device__ __forceinline__ const bf16* q_row(int r) const {
    const int i = row0 + r;
    return i < q_len ? q + i * q_tok_stride : nullptr;
  }
  __device__ __forceinline__ int lim(int r) const {
    const int i = row0 + r;
    return i < q_len ? pos + i + 1 : 0;
  }
  __device__ __forceinline__ float* out_row(int r) const {
    const int i = row0 + r;
    return i < q_len ? out + i * q_tok_stride : nullptr;
  }
  __device__ __forceinline__ float* lse_ptr(int r) const { return lse ? lse + row0 + r : nullptr; }
  __device__ __forceinline__ float* ml_ptr(int) const { return nullptr; }
};

template <int D>
__global__ void __launch_bounds__(128) prefill_mma_kernel(PrefillParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int nbh = p.c.batch * p.q_heads;
  const int bh = blockIdx.x % nbh;
  const int t = p.tiles - 1 - blockIdx.x / nbh;  // longest KV range first
  const int b = bh / p.q_heads, h = bh % p.q_heads, hk = h / p.group;

  PrefillItem<D> it;
  it.k = p.c.k + b * p.c.sb + hk * p.c.sh;
  it.v = p.c.v + b * p.c.sb + hk * p.c.sh;
  it.row_stride = p.c.sr;
  it.kv_begin = 0;
  it.kv_end = p.pos + min(p.q_len, (t + 1) * 64);
  it.partial = false;
  it.q_tok_stride = static_cast<int64_t>(p.q_heads) * D;
  const int64_t base = (static_cast<int64_t>(b) * p.q_len * p.q_heads + h) * D;
  it.q = p.q + base;
  it.out = p.out + base;
  it.lse = p.lse ? p.lse + (static_cast<int64_t>(b) * p.q_heads + h) * p.q_len : nullptr;
  it.row0 = t * 64;
  it.q_len = p.q_len;
  it.pos = p.pos;
  attn_tile_mma<D, 2>(it, p.scale_log2, smem);
}

cudaError_t launch_prefill_mma(const bf16* q, const CacheView& c, int q_heads, int q_len, int pos, float scale,
                               float* out, float* lse, cudaStream_t st, LaunchInfo& li) {
  PrefillParams p;
  p.q = q;
  p.c = c;
  p.q_heads = q_heads;
  p.group = q_heads / c.kv_heads;
  p.q_len = q_len;
  p.pos = pos;
  p.tiles = (q_len + 63) / 64;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.out = out;
  p.lse = lse;
  const unsigned grid = static_cast<unsigned>(p.tiles) * c.batch * q_heads;
  cudaError_t e;
  if (c.head_dim == 128) {
    constexpr int smem = MmaTileCfg<128, 2>::SMEM_BYTES;
    static PerDeviceOnce attr_done;
    if (!attr_done.done()) {
      e = cudaFuncSetAttribute(prefill_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(prefill_mma_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared);
      if (e != cudaSuccess) return e;
      attr_done.set();
    }
    prefill_mma_kernel<128><<<grid, 128, smem, st>>>(p);
  } else {
    constexpr int smem = MmaTileCfg<64, 2>::SMEM_BYTES;
    static PerDeviceOnce attr_done;
    if (!attr_done.done()) {
      e = cudaFuncSetAttribute(prefill_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(prefill_mma_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout,
                                 cudaSharedmemCarveoutMaxShared);
      if (e != cudaSuccess) return e;
      attr_done.set();
    }
    prefill_mma_kernel<64><<<grid, 128, smem, st>>>(p);
  }
  li.launches += 1;
  return cudaGetLastError();
}

}  // namespace jup
