// KVCache compaction after token-tree verification (paper Sec. V-A, Fig. 7 step 5: the rejected
// draft tokens are removed from the KVCache).  With a chain the accepted tokens are the first rows of
// the block and the caller only lowers the length; with a tree the accepted root-to-leaf path is
// scattered over the block's rows, and its rows move, in path order, to the front of the block:
//     row (pos_b + j)  <-  row (pos_b + accept[b][j])      j < n_accept[b], K and V, every kv head.
// One CTA per (sequence, kv head): the accepted rows are staged in shared memory before any of them is
// written, so source and destination rows may overlap.  Bit-exact 16-byte moves.
#include "host_checks.h"
#include "kernels.h"

namespace jup {

constexpr int COMPACT_MAX_ROWS = 16;

struct CompactParams {
  bf16* k;
  bf16* v;
  const int32_t* d_pos;
  const int32_t* d_accept;    // [batch][q_len]
  const int32_t* d_n_accept;  // [batch]
  int64_t sb, sh, sr;
  int kv_heads, capacity, q_len, chunks;  // chunks = D / 8
};

__global__ void __launch_bounds__(128) kv_compact_kernel(CompactParams p) {
  __shared__ uint4 stage[2 * COMPACT_MAX_ROWS * 16];  // K rows, then V rows; up to 16 pieces of 16 bytes per row
  __shared__ int src_row[COMPACT_MAX_ROWS];
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.x / p.kv_heads, h = blockIdx.x % p.kv_heads;
  const int pos = p.d_pos[b];
  int n = p.d_n_accept[b];
  n = n < 0 ? 0 : (n > p.q_len ? p.q_len : n);
  if (pos < 0 || pos > p.capacity - p.q_len) return;  // never form an address outside the cache (no overflow: q_len <= capacity)
  if (threadIdx.x < n) {
    const int a = p.d_accept[b * p.q_len + threadIdx.x];
    src_row[threadIdx.x] = (a >= 0 && a < p.q_len) ? a : -1;  // an index outside the block moves nothing
  }
  __syncthreads();
  bf16* kb = p.k + b * p.sb + h * p.sh;
  bf16* vb = p.v + b * p.sb + h * p.sh;
  for (int idx = threadIdx.x; idx < n * p.chunks; idx += blockDim.x) {
    const int j = idx / p.chunks, c = idx % p.chunks;
    if (src_row[j] < 0) continue;
    const int64_t off = static_cast<int64_t>(pos + src_row[j]) * p.sr + c * 8;
    stage[idx] = *reinterpret_cast<const uint4*>(kb + off);
    stage[COMPACT_MAX_ROWS * 16 + idx] = *reinterpret_cast<const uint4*>(vb + off);
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < n * p.chunks; idx += blockDim.x) {
    const int j = idx / p.chunks, c = idx % p.chunks;
    if (src_row[j] < 0 || src_row[j] == j) continue;
    const int64_t off = static_cast<int64_t>(pos + j) * p.sr + c * 8;
    *reinterpret_cast<uint4*>(kb + off) = stage[idx];
    *reinterpret_cast<uint4*>(vb + off) = stage[COMPACT_MAX_ROWS * 16 + idx];
  }
}

cudaError_t launch_kv_compact(const CacheView& c, int q_len, const int32_t* d_pos, const int32_t* d_accept,
                              const int32_t* d_n_accept, cudaStream_t st, LaunchInfo& li) {
  CompactParams p;
  p.k = const_cast<bf16*>(c.k);
  p.v = const_cast<bf16*>(c.v);
  p.d_pos = d_pos;
  p.d_accept = d_accept;
  p.d_n_accept = d_n_accept;
  p.sb = c.sb;
  p.sh = c.sh;
  p.sr = c.sr;
  p.kv_heads = c.kv_heads;
  p.capacity = c.capacity;
  p.q_len = q_len;
  p.chunks = c.head_dim / 8;
  static PerDeviceOnce attr_done;
  if (!attr_done.done()) {
    cudaError_t e = cudaFuncSetAttribute(kv_compact_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                         cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  li.launches += 1;
  return launch_pdl(kv_compact_kernel, dim3(static_cast<unsigned>(c.batch) * c.kv_heads), dim3(128), 0, st, p);
}

}  // namespace jup
