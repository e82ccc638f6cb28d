// Internal launch interface between the C-ABI layer (api.cu) and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace jup {

// A validated cache descriptor (strides in elements).
struct CacheView {
  const bf16* k;
  const bf16* v;
  int batch, kv_heads, capacity, head_dim;
  int64_t sb, sh, sr;
};

// The first bytes of a context's scratch hold the branch kernels' arrival counters (zero between launches);
// kernels that need scratch for data use the part behind them.
constexpr size_t SCRATCH_COUNTER_BYTES = 65536;

struct LaunchInfo {
  int sm_count;
  int launches;  // incremented by every launcher, one per kernel launch
};

// Launch with programmatic stream serialisation allowed: the kernel may be scheduled while the previous
// kernel of the stream drains; it calls pdl_wait() before touching global memory.  cluster > 1 launches
// thread-block clusters of that many consecutive CTAs.
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                      unsigned cluster, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cluster > 1) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  return launch_pdl_cluster(kernel, grid, block, smem, st, 1u, static_cast<Args&&>(args)...);
}

cudaError_t launch_kv_append(const CacheView& c, const bf16* k_new, const bf16* v_new, int n_rows, int pos,
                             const int32_t* d_pos, cudaStream_t st, LaunchInfo& li);

cudaError_t launch_prefill_mma(const bf16* q, const CacheView& c, int q_heads, int q_len, int pos, float scale,
                               float* out, float* lse, cudaStream_t st, LaunchInfo& li);

// tcgen05 / TMEM prefill kernel (head_dim 128, positive finite scale, TMA-encodable strides).
bool prefill_tc_supported(const CacheView& c, float scale);
// prefix (nullable) / prefix_len: a shared cache (batch 1) whose rows [0, prefix_len) every query row attends
// before the sequence's own rows.
// workspace: the context's scratch (used by the cluster mode for partial results; may be null).
cudaError_t launch_prefill_tc(const bf16* q, const CacheView& c, const CacheView* prefix, int prefix_len,
                              int q_heads, int q_len, int pos, float scale, float* out, float* lse, int* status,
                              void* workspace, size_t workspace_bytes, cudaStream_t st, LaunchInfo& li);

// Fused KVCache write + attention: the chunk's K/V (k_new / v_new, [batch][q_len][kv_heads][128] token-major) go into
// cache rows [pos, pos + q_len) and the chunk attends cache rows [0, pos) plus itself, in one launch.
cudaError_t launch_prefill_tc_fused(const bf16* q, const CacheView& c, const bf16* k_new, const bf16* v_new,
                                    int q_heads, int q_len, int pos, float scale, float* out, float* lse, int* status,
                                    void* workspace, size_t workspace_bytes, cudaStream_t st, LaunchInfo& li);

// Scratch needed by launch_branch for these sizes (bytes).
size_t branch_workspace_bytes(int prefix_len, int max_suffix_len, int n_branches, int q_heads, int kv_heads,
                              int q_len, int head_dim, int sm_count);

// d_tree_mask: nullptr for a chain (causal inside the draft block), else [n_branches][q_len] bit masks.
// k_new / v_new (nullable, [n_branches][q_len][kv_heads][D]): fused KVCache write -- the block's K/V are read from
// there and stored into suffix rows [L_b - q_len, L_b) by the same launch.
cudaError_t launch_branch(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                          const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len, int n_branches,
                          int q_heads, int q_len, float scale, float* out, float* lse, void* workspace,
                          cudaStream_t st, LaunchInfo& li, const bf16* k_new = nullptr, const bf16* v_new = nullptr);

// Streaming form of branch attention: clusters walk prefix + suffixes with one softmax state per row and merge
// through distributed shared memory; no scratch.  Preferred when all stacked rows of a kv head fit one 16-row tile, or
// when the (kv head, 16-row tile) units all run at once.
bool branch_stream_preferred(int n_branches, int q_heads, int kv_heads, int q_len, int sm_count);
cudaError_t launch_branch_stream(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                                 const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len,
                                 int n_branches, int q_heads, int q_len, float scale, float* out, float* lse,
                                 cudaStream_t st, LaunchInfo& li, const bf16* k_new = nullptr,
                                 const bf16* v_new = nullptr);

// Branch attention on tcgen05 / TMEM for many stacked rows per kv head (head_dim 128, positive finite scale; a
// branch's q_len x group rows must fit a 128-row tile or the group size must divide 128): units of (kv head, row
// tile) walk prefix + suffixes with one softmax state per row; the CTAs that share a unit form a thread-block
// cluster and exchange their partials through the scratch (with too little of it a unit is walked by one CTA, so
// the call never fails for lack of scratch).  Both calls need the target device current.
bool branch_tc_supported(const CacheView& suffix, int prefix_len, int max_suffix_len, int n_branches, int q_heads,
                         int q_len, float scale, int sm_count);
cudaError_t launch_branch_tc(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                             const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len,
                             int n_branches, int q_heads, int q_len, float scale, float* out, float* lse, int* status,
                             long long wait_limit, void* workspace, size_t workspace_bytes, cudaStream_t st,
                             LaunchInfo& li, const bf16* k_new = nullptr, const bf16* v_new = nullptr);

// One CTA that waits, for at most limit_cycles SM clocks, on a barrier nobody arrives at, then reports through the
// status word like any kernel whose bounded wait ran out.
cudaError_t launch_wait_probe(int* status, long long limit_cycles, cudaStream_t st, LaunchInfo& li);

// The same step for several decoder layers in one launch of the streaming kernel (at most
// kBranchMaxLayersPerLaunch per launch; more layers take further launches): every layer has its own tensors, all
// share the geometry of `prefix` / `suffix` (whose own k / v are ignored), the lengths and the scale.
constexpr int kBranchMaxLayersPerLaunch = 16;
struct BranchLayerTensors {
  const bf16* q;
  const bf16* k_new;  // nullable (all layers alike): no fused KVCache write
  const bf16* v_new;
  const bf16* pk;
  const bf16* pv;
  const bf16* sk;
  const bf16* sv;
  float* out;
  float* lse;  // nullable
};
cudaError_t launch_branch_stream_layers(const BranchLayerTensors* layers, int n_layers, const CacheView& prefix,
                                        int prefix_len, const CacheView& suffix, const int32_t* d_suffix_len,
                                        int max_suffix_len, int n_branches, int q_heads, int q_len, float scale,
                                        cudaStream_t st, LaunchInfo& li);

// Moves the accepted rows of every sequence's draft block (q_len <= 16 rows at d_pos[b]) to the front of the block.
cudaError_t launch_kv_compact(const CacheView& c, int q_len, const int32_t* d_pos, const int32_t* d_accept,
                              const int32_t* d_n_accept, cudaStream_t st, LaunchInfo& li);

// Plain read of `bytes` bytes (multiple of 16, 16-byte aligned); `out` (one word) is incremented only if the XOR of
// all words read equals a fixed constant.
cudaError_t launch_read_probe(const void* src, size_t bytes, uint32_t* out, cudaStream_t st, LaunchInfo& li);

}  // namespace jup
