// Branch attention (paper Sec. V-B: every point-extending request shares the prompt's
// KVCache; Sec. V-A step 3: q_len draft tokens verified in one pass, causal inside
// the block).
//
// Split-KV in two kinds of work items, all in one launch:
//   prefix item (kv head, prefix split, row tile): the stacked query rows of ALL
//     branches, draft tokens and heads of the group (16 or 32 per CTA) stream a slice of
//     the shared prefix, so a prefix row is fetched once per row tile instead of once per
//     branch; the four warps of a CTA split every 64-key tile by keys;
//   suffix item (branch, kv head, suffix split, row tile): that branch's rows stream a
//     slice of its own suffix, with the causal limit of each draft row.
// Each item writes an unnormalised partial (O, m, l) per row into scratch.  The partials of a
// (branch, kv head) group are merged in fixed slot order (so the result never depends on
// timing) and normalised
//   - in the same launch when a group has few rows (decode): every item takes a ticket on the
//     counters of the groups it contributed to and the CTA that takes a group's last ticket does
//     the merge; nothing waits on anything;
//   - by a second, fully parallel launch when a group has many rows (draft verification with
//     grouped heads), where one CTA per group would serialise too much work at the tail.
// Scratch layout: [64 KiB of int32 counters, one per (branch, kv head), zero between calls]
// [O partials][(m, l) partials].  The merging CTA puts each counter back to zero.
#include "attn_keysplit.cuh"
#include "host_checks.h"
#include "kernels.h"

namespace jup {

constexpr size_t BRANCH_COUNTER_BYTES = SCRATCH_COUNTER_BYTES;  // fixed block at the start of the scratch
constexpr int BRANCH_MAX_GROUPS = static_cast<int>(BRANCH_COUNTER_BYTES / sizeof(int));

struct BranchPlan {
  int tile_rows;                           // stacked query rows per CTA: 16 or 32
  int one_shot;                            // items of <= 128 keys fetched whole (few rows: pure streaming)
  int row_tiles_p, splits_p, split_len_p;  // prefix
  int row_tiles_s, splits_s, split_len_s;  // suffix
  int items_p, items_s, slots;
};

static int ceil_div(int a, int b) { return (a + b - 1) / b; }

static BranchPlan make_plan(int prefix_len, int max_suffix_len, int n_branches, int q_heads, int kv_heads, int q_len,
                            int sm_count) {
  BranchPlan pl;
  const int G = q_heads / kv_heads;
  const int rows_p = n_branches * q_len * G, rows_s = q_len * G;
  pl.tile_rows = rows_p <= 16 ? 16 : 32;
  pl.row_tiles_p = ceil_div(rows_p, pl.tile_rows);
  pl.row_tiles_s = ceil_div(rows_s, pl.tile_rows);
  // keys per work item.  With at most 16 stacked rows the job is pure K/V streaming: items of 128
  // keys, fetched whole, three CTAs per SM.  Otherwise the whole job is spread over about three
  // CTAs per SM with at least 128 keys each, streamed through a ring.
  const int64_t work = static_cast<int64_t>(prefix_len) * kv_heads * pl.row_tiles_p +
                       static_cast<int64_t>(max_suffix_len) * n_branches * kv_heads * pl.row_tiles_s;
  int64_t target = (work / (3 * static_cast<int64_t>(sm_count)) + 63) / 64 * 64;
  if (target < 128) target = 128;
  if (target > (1 << 20)) target = 1 << 20;
  pl.one_shot = pl.tile_rows == 16;
  const int tgt = pl.one_shot ? 128 : static_cast<int>(target);
  if (prefix_len > 0) {
    pl.splits_p = ceil_div(prefix_len, tgt);
    pl.split_len_p = ceil_div(ceil_div(prefix_len, pl.splits_p), 64) * 64;
    pl.splits_p = ceil_div(prefix_len, pl.split_len_p);
  } else {
    pl.split_len_p = 64;
    pl.splits_p = 0;
  }
  pl.splits_s = ceil_div(max_suffix_len, tgt);
  pl.split_len_s = ceil_div(ceil_div(max_suffix_len, pl.splits_s), 64) * 64;
  pl.splits_s = ceil_div(max_suffix_len, pl.split_len_s);
  pl.items_p = kv_heads * pl.splits_p * pl.row_tiles_p;
  pl.items_s = n_branches * kv_heads * pl.splits_s * pl.row_tiles_s;
  pl.slots = pl.splits_p + pl.splits_s;
  return pl;
}

size_t branch_workspace_bytes(int prefix_len, int max_suffix_len, int n_branches, int q_heads, int kv_heads,
                              int q_len, int head_dim, int sm_count) {
  const BranchPlan pl = make_plan(prefix_len, max_suffix_len, n_branches, q_heads, kv_heads, q_len, sm_count);
  if (static_cast<int64_t>(n_branches) * kv_heads > BRANCH_MAX_GROUPS) return ~static_cast<size_t>(0);
  const size_t rows = static_cast<size_t>(n_branches) * q_len * q_heads;
  return BRANCH_COUNTER_BYTES + rows * pl.slots * (static_cast<size_t>(head_dim) + 2) * sizeof(float);
}

struct BranchParams {
  const bf16* q;
  CacheView prefix, suffix;
  const int32_t* d_suffix_len;
  const uint32_t* tree_mask;  // nullable: [n_branches][q_len], bit j of entry (b, i): draft row i sees draft row j
  // fused KVCache write (nullable): this step's K/V block, [n_branches][q_len][kv_heads][D]; its rows are read
  // from here instead of the suffix cache and written to suffix rows [L_b - q_len, L_b)
  const bf16* k_new;
  const bf16* v_new;
  int prefix_len, max_suffix_len, n_branches, q_heads, group, q_len;
  BranchPlan pl;
  float scale_log2;
  int* counters;   // [n_branches][kv_heads], zero on entry and on exit
  float* o_part;   // [rows][slots][D]
  float* ml_part;  // [rows][slots][2]
  float* out;
  float* lse;
};

template <int D>
struct BranchItem {
  const bf16* k;
  const bf16* v;
  int64_t row_stride;
  int kv_begin, kv_end;
  bool partial;
  const bf16* q;
  float* o_part;
  float* ml_part;
  int R0, R_count;          // first stacked row of this tile, number of stacked rows in the item's row space
  int n, G, q_heads, hk;    // draft rows, group size
  int b_fixed;              // >= 0: suffix item of that branch; -1: prefix item (row index carries the branch)
  int lim_base;             // suffix: L_b - n + 1 (row i sees keys < lim_base + i); prefix: prefix_len
  int hist;                 // first key of the draft block when a tree mask applies, else INT_MAX
  const uint32_t* tmask_b;  // tree masks of this branch (q_len entries) or nullptr
  int new_begin;            // first key that comes from k_new / v_new (INT_MAX: none)
  int64_t new_stride;       // row stride of k_new / v_new
  const bf16* k_new;
  const bf16* v_new;
  bf16* k_cache;            // this item's cache rows, writable (writer items only)
  bf16* v_cache;
  bool writer;              // stores the new rows it loads into the cache
  int slot, slots;
  __device__ __forceinline__ bool decode(int r, int& b, int& i, int& g) const {
    const int R = R0 + r;
    if (R >= R_count) return false;
    g = R % G;
    const int t = R / G;
    i = t % n;
    b = b_fixed >= 0 ? b_fixed : t / n;
    return true;
  }
  __device__ __forceinline__ int64_t rowid(int b, int i, int g) const {
    return (static_cast<int64_t>(b) * n + i) * q_heads + hk * G + g;
  }
  __device__ __forceinline__ const bf16* q_row(int r) const {
    int b, i, g;
    return decode(r, b, i, g) ? q + rowid(b, i, g) * D : nullptr;
  }
  __device__ __forceinline__ int lim(int r) const {
    int b, i, g;
    if (!decode(r, b, i, g)) return 0;
    if (tmask_b) return lim_base + n - 1;  // tree: every row of the block is a candidate, the mask decides
    return b_fixed >= 0 ? lim_base + i : lim_base;
  }
  __device__ __forceinline__ uint32_t tmask(int r) const {
    int b, i, g;
    if (!tmask_b || !decode(r, b, i, g)) return 0xffffffffu;
    return tmask_b[i];
  }
  __device__ __forceinline__ float* out_row(int r) const {
    int b, i, g;
    return decode(r, b, i, g) ? o_part + (rowid(b, i, g) * slots + slot) * D : nullptr;
  }
  __device__ __forceinline__ float* lse_ptr(int) const { return nullptr; }
  __device__ __forceinline__ float* ml_ptr(int r) const {
    int b, i, g;
    return decode(r, b, i, g) ? ml_part + (rowid(b, i, g) * slots + slot) * 2 : nullptr;
  }
};

__device__ __forceinline__ int clamp_len(int L, int lo, int hi) { return L < lo ? lo : (L > hi ? hi : L); }

// Merge the partials of row r (draft token r / G, head r % G of the group) of group (branch b, kv
// head hk); executed by one warp.  Lanes first
// fetch the (m, l) pairs of 32 slots at a time, the row maximum and the weights follow from warp
// reductions, then the O partials are accumulated in slot order with the loads of four slots in
// flight.  The order of the floating-point sums is fixed, whichever CTA does the merge.
template <int D>
__device__ __forceinline__ void merge_row(const BranchParams& p, int b, int hk, int r) {
  const int lane = threadIdx.x & 31;
  const int L = clamp_len(p.d_suffix_len[b], p.q_len, p.max_suffix_len);
  const int slots = p.pl.slots, sp = p.pl.splits_p;
  constexpr int V = D / 32;
  {
    const int i = r / p.group, g = r % p.group, h = hk * p.group + g;
    const int64_t row = (static_cast<int64_t>(b) * p.q_len + i) * p.q_heads + h;
    const float2* ml = reinterpret_cast<const float2*>(p.ml_part + row * slots * 2);
    auto slot_ml = [&](int s) {  // (m, l) of slot s, (-inf, 0) if the slot does not exist for this branch
      const bool valid = s < slots && (s < sp || (s - sp) * p.pl.split_len_s < L);
      return valid ? __ldcg(ml + s) : make_float2(-INFINITY, 0.f);
    };
    float M = -INFINITY;
    for (int base = 0; base < slots; base += 32) M = fmaxf(M, slot_ml(base + lane).x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float acc[V];
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] = 0.f;
    float Lsum = 0.f;
    for (int base = 0; base < slots; base += 32) {
      const float2 mine = slot_ml(base + lane);
      const float w_mine = mine.x == -INFINITY ? 0.f : fast_exp2(mine.x - M);
      float lw = mine.y * w_mine;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o);
      Lsum += lw;
      const int cnt = min(32, slots - base);
      const float* op = p.o_part + (row * slots + base) * D + lane * V;
      for (int s0 = 0; s0 < cnt; s0 += 4) {
        float w[4];
        float vbuf[4][V];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          w[u] = __shfl_sync(0xffffffffu, w_mine, (s0 + u) & 31);
          const bool on = (s0 + u < cnt) && w[u] != 0.f;
          if (!on) w[u] = 0.f;
          if constexpr (V == 4) {
            const float4 v = on ? __ldcg(reinterpret_cast<const float4*>(op + (s0 + u) * D)) : make_float4(0, 0, 0, 0);
            vbuf[u][0] = v.x;
            vbuf[u][1] = v.y;
            vbuf[u][2] = v.z;
            vbuf[u][3] = v.w;
          } else {
            const float2 v = on ? __ldcg(reinterpret_cast<const float2*>(op + (s0 + u) * D)) : make_float2(0, 0);
            vbuf[u][0] = v.x;
            vbuf[u][1] = v.y;
          }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int j = 0; j < V; ++j) acc[j] += vbuf[u][j] * w[u];
      }
    }
    const float inv = 1.f / Lsum;
    float* o = p.out + row * D + lane * V;
    if constexpr (V == 4)
      *reinterpret_cast<float4*>(o) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
    else
      *reinterpret_cast<float2*>(o) = make_float2(acc[0] * inv, acc[1] * inv);
    if (p.lse && lane == 0)
      p.lse[(static_cast<int64_t>(b) * p.q_heads + h) * p.q_len + i] = (M + log2f(Lsum)) * 0.69314718055994530942f;
  }
}

template <int D, int MT, int STAGES, bool FUSED_MERGE>
__global__ void __launch_bounds__(128) branch_attn_kernel(BranchParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ int s_done[40];  // [0] = count, then the branches whose group this CTA completed
  pdl_wait();
  BranchItem<D> it;
  it.partial = true;
  it.q = p.q;
  it.o_part = p.o_part;
  it.ml_part = p.ml_part;
  it.n = p.q_len;
  it.G = p.group;
  it.q_heads = p.q_heads;
  it.slots = p.pl.slots;
  it.new_begin = 0x7fffffff;
  it.new_stride = 0;
  it.k_new = it.v_new = nullptr;
  it.k_cache = it.v_cache = nullptr;
  it.writer = false;
  const int rows_per_branch = p.q_len * p.group;
  int x = blockIdx.x;
  int b_first, b_last, hk;  // the groups (b, hk), b_first <= b <= b_last, this item contributes to
  if (x < p.pl.items_p) {
    const int rt = x % p.pl.row_tiles_p;
    x /= p.pl.row_tiles_p;
    const int sp = x % p.pl.splits_p;
    hk = x / p.pl.splits_p;
    it.hk = hk;
    it.k = p.prefix.k + hk * p.prefix.sh;
    it.v = p.prefix.v + hk * p.prefix.sh;
    it.row_stride = p.prefix.sr;
    it.kv_begin = sp * p.pl.split_len_p;
    it.kv_end = min(p.prefix_len, it.kv_begin + p.pl.split_len_p);
    it.R0 = rt * (16 * MT);
    it.R_count = p.n_branches * rows_per_branch;
    it.b_fixed = -1;
    it.lim_base = p.prefix_len;
    it.hist = 0x7fffffff;
    it.tmask_b = nullptr;
    it.slot = sp;
    b_first = it.R0 / rows_per_branch;
    b_last = (min(it.R0 + 16 * MT, it.R_count) - 1) / rows_per_branch;
  } else {
    x -= p.pl.items_p;
    const int rt = x % p.pl.row_tiles_s;
    x /= p.pl.row_tiles_s;
    const int ss = x % p.pl.splits_s;
    x /= p.pl.splits_s;
    hk = x % p.suffix.kv_heads;
    const int b = x / p.suffix.kv_heads;
    const int L = clamp_len(p.d_suffix_len[b], p.q_len, p.max_suffix_len);
    it.kv_begin = ss * p.pl.split_len_s;
    if (it.kv_begin >= L) return;  // not counted: the expected ticket count below uses the same test
    it.kv_end = min(L, it.kv_begin + p.pl.split_len_s);
    it.hk = hk;
    it.k = p.suffix.k + b * p.suffix.sb + hk * p.suffix.sh;
    it.v = p.suffix.v + b * p.suffix.sb + hk * p.suffix.sh;
    it.row_stride = p.suffix.sr;
    it.R0 = rt * (16 * MT);
    it.R_count = rows_per_branch;
    it.b_fixed = b;
    it.lim_base = L - p.q_len + 1;
    it.tmask_b = p.tree_mask ? p.tree_mask + static_cast<int64_t>(b) * p.q_len : nullptr;
    it.hist = p.tree_mask ? L - p.q_len : 0x7fffffff;
    it.slot = p.pl.splits_p + ss;
    if (p.k_new) {  // every key belongs to one split: the first row tile of that split writes it
      const int64_t noff = (static_cast<int64_t>(b) * p.q_len * p.suffix.kv_heads + hk) * D;
      it.new_begin = L - p.q_len;
      it.new_stride = static_cast<int64_t>(p.suffix.kv_heads) * D;
      it.k_new = p.k_new + noff;
      it.v_new = p.v_new + noff;
      it.k_cache = const_cast<bf16*>(it.k);
      it.v_cache = const_cast<bf16*>(it.v);
      it.writer = rt == 0;
    }
    b_first = b_last = b;
  }
  attn_tile_keysplit<D, MT, STAGES>(it, p.scale_log2, smem);
  pdl_launch_dependents();
  if constexpr (!FUSED_MERGE) return;

  // ---- tickets: the partials above must be visible before the ticket is
  __threadfence();
  __syncthreads();
  if (threadIdx.x < 32) {  // one lane per group this item contributed to (at most 33: two rounds)
    int n_done = 0;
    for (int b0 = b_first; b0 <= b_last; b0 += 32) {
      const int b = b0 + static_cast<int>(threadIdx.x);
      bool done = false;
      if (b <= b_last) {
        // CTAs that contribute to group (b, hk): prefix splits x row tiles overlapping the branch's rows,
        // plus the suffix splits that start below its length x suffix row tiles
        const int lo = b * rows_per_branch, hi = lo + rows_per_branch - 1;
        const int tiles = hi / (16 * MT) - lo / (16 * MT) + 1;
        const int L = clamp_len(p.d_suffix_len[b], p.q_len, p.max_suffix_len);
        const int expected =
            p.pl.splits_p * tiles + ((L + p.pl.split_len_s - 1) / p.pl.split_len_s) * p.pl.row_tiles_s;
        int* cnt = p.counters + b * p.suffix.kv_heads + hk;
        done = atomicAdd(cnt, 1) + 1 == expected;
        if (done) *cnt = 0;  // every contributor has taken its ticket: ready for the next call
      }
      const unsigned mask = __ballot_sync(0xffffffffu, done);
      if (done) s_done[1 + n_done + __popc(mask & ((1u << threadIdx.x) - 1u))] = b;
      n_done += __popc(mask);
    }
    if (threadIdx.x == 0) s_done[0] = n_done;
    __threadfence();  // the others' partials are read after this
  }
  __syncthreads();
  const int n_done = s_done[0];
  // the rows of all completed groups, dealt round-robin to the four warps
  for (int idx = threadIdx.x >> 5; idx < n_done * rows_per_branch; idx += 4)
    merge_row<D>(p, s_done[1 + idx / rows_per_branch], hk, idx % rows_per_branch);
}

// Second launch of the two-launch form: one warp per output row; blockIdx.x = group, blockIdx.y = 4 rows.
template <int D>
__global__ void __launch_bounds__(128) branch_merge_kernel(BranchParams p) {
  pdl_launch_dependents();
  pdl_wait();
  const int r = blockIdx.y * 4 + (threadIdx.x >> 5);
  if (r < p.q_len * p.group) merge_row<D>(p, blockIdx.x / p.suffix.kv_heads, blockIdx.x % p.suffix.kv_heads, r);
}

template <int D, int MT, int STAGES, bool FUSED_MERGE>
static cudaError_t launch_branch_d(const BranchParams& p, cudaStream_t st, LaunchInfo& li) {
  constexpr int smem = KeySplitCfg<D, MT, STAGES>::SMEM_BYTES;
  static PerDeviceOnce attr_done;
  if (!attr_done.done()) {
    cudaError_t e = cudaFuncSetAttribute(branch_attn_kernel<D, MT, STAGES, FUSED_MERGE>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(branch_attn_kernel<D, MT, STAGES, FUSED_MERGE>,
                               cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess && !FUSED_MERGE)
      e = cudaFuncSetAttribute(branch_merge_kernel<D>, cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  const unsigned grid = static_cast<unsigned>(p.pl.items_p + p.pl.items_s);
  cudaError_t e = launch_pdl(branch_attn_kernel<D, MT, STAGES, FUSED_MERGE>, dim3(grid), dim3(128), smem, st, p);
  li.launches += 1;
  if (FUSED_MERGE || e != cudaSuccess) return e;
  const dim3 mgrid(static_cast<unsigned>(p.n_branches * p.suffix.kv_heads),
                   static_cast<unsigned>((p.q_len * p.group + 3) / 4));
  li.launches += 1;
  return launch_pdl(branch_merge_kernel<D>, mgrid, dim3(128), 0, st, p);
}

cudaError_t launch_branch(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                          const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len, int n_branches,
                          int q_heads, int q_len, float scale, float* out, float* lse, void* workspace,
                          cudaStream_t st, LaunchInfo& li, const bf16* k_new, const bf16* v_new) {
  BranchParams p;
  p.q = q;
  p.k_new = k_new;
  p.v_new = v_new;
  p.tree_mask = d_tree_mask;
  p.prefix = prefix;
  p.suffix = suffix;
  p.d_suffix_len = d_suffix_len;
  p.prefix_len = prefix_len;
  p.max_suffix_len = max_suffix_len;
  p.n_branches = n_branches;
  p.q_heads = q_heads;
  p.group = q_heads / suffix.kv_heads;
  p.q_len = q_len;
  p.pl = make_plan(prefix_len, max_suffix_len, n_branches, q_heads, suffix.kv_heads, q_len, li.sm_count);
  p.scale_log2 = scale * 1.4426950408889634f;
  const size_t rows = static_cast<size_t>(n_branches) * q_len * q_heads;
  p.counters = static_cast<int*>(workspace);
  p.o_part = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + BRANCH_COUNTER_BYTES);
  p.ml_part = p.o_part + rows * p.pl.slots * suffix.head_dim;
  p.out = out;
  p.lse = lse;
  if (suffix.head_dim == 128)
    return p.pl.one_shot ? launch_branch_d<128, 1, 0, true>(p, st, li) : launch_branch_d<128, 2, 3, false>(p, st, li);
  return p.pl.one_shot ? launch_branch_d<64, 1, 0, true>(p, st, li) : launch_branch_d<64, 2, 3, false>(p, st, li);
}

}  // namespace jup
