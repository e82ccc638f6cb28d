// KVCache write (paper Sec. II-A; Sec. V-A step 3): token-major new K/V rows are
// moved bit-exactly into head-major cache rows [pos_b, pos_b + n).  Pure data
// movement, HBM-bound: every thread moves 16-byte chunks with 128-bit loads/stores.
#include "host_checks.h"
#include "kernels.h"

namespace jup {

struct AppendParams {
  const uint4* k_new;
  const uint4* v_new;
  bf16* k;
  bf16* v;
  const int32_t* d_pos;
  int64_t sb, sh, sr;
  int batch, kv_heads, capacity, n_rows, pos, chunks;  // chunks = D / 8
  int64_t total;                                        // batch * n_rows * kv_heads * chunks
};

__global__ void __launch_bounds__(256) kv_append_kernel(AppendParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < p.total; idx += stride) {
    const int c = static_cast<int>(idx % p.chunks);
    int64_t r = idx / p.chunks;
    const int h = static_cast<int>(r % p.kv_heads);
    r /= p.kv_heads;
    const int t = static_cast<int>(r % p.n_rows);
    const int b = static_cast<int>(r / p.n_rows);
    const int pos = p.d_pos ? p.d_pos[b] : p.pos;
    if (pos < 0 || pos > p.capacity - p.n_rows) continue;  // never form an address outside the cache (no overflow: n_rows <= capacity)
    const int64_t dst = b * p.sb + h * p.sh + static_cast<int64_t>(pos + t) * p.sr + c * 8;
    const uint4 kk = p.k_new[idx];
    const uint4 vv = p.v_new[idx];
    *reinterpret_cast<uint4*>(p.k + dst) = kk;
    *reinterpret_cast<uint4*>(p.v + dst) = vv;
  }
}

cudaError_t launch_kv_append(const CacheView& c, const bf16* k_new, const bf16* v_new, int n_rows, int pos,
                             const int32_t* d_pos, cudaStream_t st, LaunchInfo& li) {
  AppendParams p;
  p.k_new = reinterpret_cast<const uint4*>(k_new);
  p.v_new = reinterpret_cast<const uint4*>(v_new);
  p.k = const_cast<bf16*>(c.k);
  p.v = const_cast<bf16*>(c.v);
  p.d_pos = d_pos;
  p.sb = c.sb;
  p.sh = c.sh;
  p.sr = c.sr;
  p.batch = c.batch;
  p.kv_heads = c.kv_heads;
  p.capacity = c.capacity;
  p.n_rows = n_rows;
  p.pos = pos;
  p.chunks = c.head_dim / 8;
  p.total = static_cast<int64_t>(c.batch) * n_rows * c.kv_heads * p.chunks;
  if (p.total == 0) return cudaSuccess;
  const int threads = 256;
  int64_t blocks = (p.total + threads - 1) / threads;
  const int64_t cap = static_cast<int64_t>(li.sm_count) * 16;
  if (blocks > cap) blocks = cap;
  // Keep the SM's shared-memory carve-out where the attention kernels (which follow every append)
  // need it: a launch that prefers a different L1/shared split makes the SMs reconfigure in between.
  static PerDeviceOnce attr_done;
  if (!attr_done.done()) {
    cudaError_t e = cudaFuncSetAttribute(kv_append_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  li.launches += 1;
  return launch_pdl(kv_append_kernel, dim3(static_cast<unsigned>(blocks)), dim3(threads), 0, st, p);
}

}  // namespace jup
