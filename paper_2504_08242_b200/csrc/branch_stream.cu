// Branch attention, streaming form (paper Sec. V-B: the prompt's KVCache is shared by every
// point-extending request; Sec. V-A step 3: the draft block is verified in one pass).
//
// A unit = (kv head, tile of 16 stacked query rows); the stacked rows of a kv head are all
// (branch, draft token, head of the group) rows in that order.  Every row belongs to exactly
// one branch, and the keys it may see are the shared prefix plus that branch's suffix, so the
// row keeps ONE running softmax state (O, m, l) while the unit walks the concatenation
//     prefix | suffix of the tile's first branch | ... | suffix of its last branch
// in chunks of 16 keys: a prefix chunk is visible to every row, a suffix chunk only to the
// rows of its branch (up to the row's causal limit or tree mask).  The prefix is therefore
// fetched once per unit for all branches of the tile.
//
// A thread-block cluster of `cluster` CTAs shares a unit.  The prefix chunks are cut into equal
// contiguous ranges, one per CTA, and so are the suffix chunks; a CTA deals its chunks round-robin
// to its warps (the suffix deal starts where the prefix deal stopped).  The prefix share does not
// depend on the device-side lengths, so its first loads are in flight while the lengths arrive.
// Each warp is an independent stream: its own cp.async ring of 16-key K/V tiles, no CTA-wide
// barrier in the loop, mma.sync for Q K^T and P V with fp32 online softmax.  At the end the
// warps' states are merged in shared memory and each CTA pushes its partial of row t into the
// shared memory of CTA t % cluster (distributed shared memory), which merges the cluster's
// partials in rank order after ONE cluster barrier -- no global scratch, no atomics, no second
// launch, and the result does not depend on timing.
//
// Fused KVCache write: with k_new / v_new the rows of this step's block are read from there
// (they are not in the cache yet) and the warp that fetched them stores them into the suffix
// rows [L_b - q_len, L_b) from shared memory.
#include <algorithm>

#include "host_checks.h"
#include "kernels.h"
#include "tc_common.cuh"

namespace jup {

struct StreamParams {
  const bf16* q;
  CacheView prefix, suffix;
  const int32_t* d_suffix_len;
  const uint32_t* tree_mask;  // nullable: [n_branches][q_len] ancestor bit masks of the draft block
  const bf16* k_new;          // nullable: [n_branches][q_len][kv_heads][D]
  const bf16* v_new;
  int prefix_len, max_suffix_len, n_branches, q_heads, group, q_len;
  int row_tiles;  // 16-row tiles per kv head
  int cluster;    // CTAs per unit: 1, 2, 4 or 8
  int cluster_log2;
  float scale_log2;
  float* out;
  float* lse;
};

// Several independent problems of the same geometry and lengths (the decoder layers of a step) in one launch:
// blockIdx.y picks the problem, whose tensors replace the ones in StreamParams.
struct StreamLayerPtrs {
  const bf16* q;
  const bf16* k_new;
  const bf16* v_new;
  const bf16* pk;
  const bf16* pv;
  const bf16* sk;
  const bf16* sv;
  float* out;
  float* lse;
};
struct StreamLayers {
  int n;  // 0: a plain launch, the tensors of StreamParams are used
  StreamLayerPtrs l[kBranchMaxLayersPerLaunch];
};

template <int D, int NW, int ST>
struct StreamCfg {
  static constexpr int ROWS = 16;
  static constexpr int THREADS = NW * 32;
  static constexpr int CH = D / 8;                 // 16-byte pieces per K/V row
  static constexpr int TILE_BYTES = 16 * D * 2;    // 16 keys of K (or of V)
  static constexpr int SLOT_BYTES = 2 * TILE_BYTES;
  static constexpr int RING_BYTES = ST * SLOT_BYTES;  // per warp
  static constexpr int Q_BYTES = ROWS * D * 2;
  static constexpr int OSTRIDE = D + 4;  // floats per row of a partial (bank-conflict-free float2 stores)
  static constexpr int PART_BYTES = ROWS * OSTRIDE * 4;  // a partial: per row D floats of O, then (m, l)
  static_assert(ST >= 2, "the ring needs two slots");
  static_assert(PART_BYTES <= RING_BYTES, "a warp's partial is staged in its own ring");
  // [Q][partials received from the cluster: (owned row, source CTA)][NW rings]
  static constexpr int SMEM_BYTES = Q_BYTES + PART_BYTES + NW * RING_BYTES;
};

// Launch shape: warps per CTA, ring slots per warp, CTAs that fit one SM with that much shared memory.
constexpr int kStreamWarps = 8, kStreamStages = 2, kStreamCtasPerSm = 1;

__device__ __forceinline__ void st_cluster_f4(uint32_t addr, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};\n" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
               : "memory");
}
__device__ __forceinline__ void st_cluster_f2(uint32_t addr, float2 v) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};\n" ::"r"(addr), "f"(v.x), "f"(v.y) : "memory");
}

__device__ __forceinline__ int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

template <int D, int NW, int ST>
__global__ void __launch_bounds__(NW * 32, kStreamCtasPerSm)
branch_stream_kernel(const StreamParams p_in, const __grid_constant__ StreamLayers layers) {
  StreamParams p = p_in;
  if (layers.n > 0) {
    const StreamLayerPtrs& l = layers.l[blockIdx.y];
    p.q = l.q;
    p.k_new = l.k_new;
    p.v_new = l.v_new;
    p.prefix.k = l.pk;
    p.prefix.v = l.pv;
    p.suffix.k = l.sk;
    p.suffix.v = l.sv;
    p.out = l.out;
    p.lse = l.lse;
  }
  using Cfg = StreamCfg<D, NW, ST>;
  constexpr int CH = Cfg::CH;
  constexpr unsigned FULL = 0xffffffffu;
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
  const uint32_t sQ = smem_u32(smem);
  const uint32_t sRecv = sQ + Cfg::Q_BYTES;
  const uint32_t sRing0 = sRecv + Cfg::PART_BYTES;
  const uint32_t sRing = sRing0 + warp * Cfg::RING_BYTES;

  const int csize = p.cluster;
  const int clg = p.cluster_log2;  // csize is a power of two
  const int unit = blockIdx.x >> clg, rank = blockIdx.x & (csize - 1);  // clusters are consecutive CTAs along x
  const int rt = unit % p.row_tiles, hk = unit / p.row_tiles;
  const int n = p.q_len, G = p.group, nG = n * G;
  const int rows_total = p.n_branches * nG;
  const int R0 = rt * 16;
  const int nvalid = min(16, rows_total - R0);
  const int b_first = R0 / nG;
  const int nb = (R0 + nvalid - 1) / nG - b_first + 1;  // branches with a row in this tile (<= 16)
  const int P = p.prefix_len;
  const bool tree = p.tree_mask != nullptr;
  const bool fused = p.k_new != nullptr;

  // ---- everything that needs no memory comes before the dependency wait: the prefix share of this CTA and warp,
  // where this thread's pieces of the Q tile come from, which rows this lane accumulates
  const int pchunks = (P + 15) >> 4;
  const int pc0 = (rank * pchunks) >> clg;
  const int pc1 = ((rank + 1) * pchunks) >> clg;
  const int npre = pc1 - pc0 > warp ? (pc1 - pc0 - warp + NW - 1) / NW : 0;
  const int warp_s = (warp - (pc1 - pc0) % NW + NW) % NW;  // this warp's place in the suffix deal
  constexpr int QI = (16 * CH + Cfg::THREADS - 1) / Cfg::THREADS;
  const bf16* q_src[QI];
  uint32_t q_dst[QI];
#pragma unroll
  for (int u = 0; u < QI; ++u) {
    const int idx = tid + u * Cfg::THREADS;
    const int row = idx / CH, c = idx % CH;
    const int R = R0 + row;
    const bool valid = idx < 16 * CH && R < rows_total;
    const int gg = R % G, t = R / G, b = t / n, i = t % n;
    q_src[u] = valid ? p.q + ((static_cast<int64_t>(b) * n + i) * p.q_heads + hk * G + gg) * D + c * 8 : nullptr;
    q_dst[u] = idx < 16 * CH ? sQ + tile_off<D>(row, c) : 0u;
  }
  int r_j[2], r_i[2], r_b[2];  // the two rows of this lane (mma accumulator layout: rows g and g + 8)
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int R = R0 + g + h * 8;
    const bool valid = R < rows_total;
    const int t = R / G;
    r_b[h] = t / n;
    r_i[h] = t % n;
    r_j[h] = valid ? r_b[h] - b_first : -1;  // branch as a lane index, or -1
  }

  // every CTA of the cluster is running before anybody writes into a peer's shared memory: arrive
  // here, wait just before the push at the end
  asm volatile("barrier.cluster.arrive.relaxed.aligned;\n" ::: "memory");
  pdl_wait();

  // ---- suffix lengths: lane j holds branch b_first + j; used only after the first loads are issued
  int L_mine = lane < nb ? __ldg(p.d_suffix_len + b_first + lane) : 0;
  // ---- Q tile
#pragma unroll
  for (int u = 0; u < QI; ++u)
    if (q_dst[u]) cp_async16(q_dst[u], q_src[u] ? q_src[u] : p.q, q_src[u] != nullptr);
  cp_async_commit();

  // ---- chunk -> segment.  All lanes of the warp call these with the same chunk index.
  struct Seg {
    const bf16* k;
    const bf16* v;
    int64_t stride;
    int key0, len, j;   // first key of the chunk, segment length, branch lane index (-1: prefix)
    int new_begin;      // first key that is read from k_new / v_new (INT_MAX: none)
    const bf16* k_new;
    const bf16* v_new;
  };
  int cum_end = 0, sc0 = 0, nsuf = 0;  // set once the lengths are known
  // chunk jj of this warp: jj < npre is a prefix chunk, the rest are suffix chunks
  auto segment = [&](int jj) {
    Seg s;
    s.new_begin = 0x7fffffff;
    s.k_new = s.v_new = nullptr;
    if (jj < npre) {
      s.j = -1;
      s.key0 = (pc0 + warp + jj * NW) * 16;
      s.len = P;
      s.k = p.prefix.k + hk * p.prefix.sh;
      s.v = p.prefix.v + hk * p.prefix.sh;
      s.stride = p.prefix.sr;
      return s;
    }
    const int c = sc0 + warp_s + (jj - npre) * NW;
    const int sj = __popc(__ballot_sync(FULL, lane < nb && cum_end <= c));
    const int prev_end = __shfl_sync(FULL, cum_end, sj > 0 ? sj - 1 : 0);
    const int Lj = __shfl_sync(FULL, L_mine, sj < 32 ? sj : 0);
    const int b = b_first + sj;
    s.j = sj;
    s.key0 = (c - (sj > 0 ? prev_end : 0)) * 16;
    s.len = Lj;
    s.k = p.suffix.k + b * p.suffix.sb + hk * p.suffix.sh;
    s.v = p.suffix.v + b * p.suffix.sb + hk * p.suffix.sh;
    s.stride = p.suffix.sr;
    if (fused) {
      const int64_t noff = (static_cast<int64_t>(b) * n * p.suffix.kv_heads + hk) * D;
      s.new_begin = Lj - n;
      s.k_new = p.k_new + noff;
      s.v_new = p.v_new + noff;
    }
    return s;
  };
  auto load_chunk = [&](int jj) {
    const Seg s = segment(jj);
    const uint32_t sK = sRing + (jj % ST) * Cfg::SLOT_BYTES, sV = sK + Cfg::TILE_BYTES;
    const int64_t nstride = static_cast<int64_t>(p.suffix.kv_heads) * D;
    if (s.key0 + 16 <= s.new_begin) {
#pragma unroll
      for (int i = 0; i < 16 * CH / 32; ++i) {
        const int idx = lane + i * 32;
        const int row = idx / CH, c = idx % CH;
        const bool ok = s.key0 + row < s.len;
        const int64_t off = ok ? static_cast<int64_t>(s.key0 + row) * s.stride + c * 8 : 0;
        cp_async16(sK + tile_off<D>(row, c), s.k + off, ok);
        cp_async16(sV + tile_off<D>(row, c), s.v + off, ok);
      }
    } else {  // the chunk holds rows of this step's block
#pragma unroll
      for (int i = 0; i < 16 * CH / 32; ++i) {
        const int idx = lane + i * 32;
        const int row = idx / CH, c = idx % CH;
        const int key = s.key0 + row;
        const bool ok = key < s.len;
        const bool fresh = ok && key >= s.new_begin;
        const int64_t off = !ok ? 0
                                : (fresh ? static_cast<int64_t>(key - s.new_begin) * nstride
                                         : static_cast<int64_t>(key) * s.stride) + c * 8;
        cp_async16(sK + tile_off<D>(row, c), (fresh ? s.k_new : s.k) + off, ok);
        cp_async16(sV + tile_off<D>(row, c), (fresh ? s.v_new : s.v) + off, ok);
      }
    }
  };

  // ---- the ring is filled before anything is computed, one cp.async group per chunk, in chunk order: first the
  // prefix chunks, which need no length
#pragma unroll
  for (int s = 0; s < ST; ++s)
    if (s < npre) {
      load_chunk(s);
      cp_async_commit();
    }

  L_mine = lane < nb ? clampi(L_mine, n, p.max_suffix_len) : 0;
  {
    int cum = (L_mine + 15) >> 4;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(FULL, cum, o);
      if (lane >= o) cum += t;
    }
    cum_end = cum;  // one past the last suffix chunk of this lane's branch
    const int Ns = __shfl_sync(FULL, cum, 31);
    sc0 = (rank * Ns) >> clg;
    const int sc1 = ((rank + 1) * Ns) >> clg;
    nsuf = sc1 - sc0 > warp_s ? (sc1 - sc0 - warp_s + NW - 1) / NW : 0;
  }
  const int nmine = npre + nsuf;
#pragma unroll
  for (int s = 0; s < ST; ++s)
    if (s >= npre) {
      if (s < nmine) load_chunk(s);
      cp_async_commit();
    }

  // ---- causal limit inside the branch's suffix (or the block's end with a tree mask) and tree masks of the rows
  int r_lim[2];
  uint32_t r_tm[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int Lb = __shfl_sync(FULL, L_mine, r_j[h] < 0 ? 0 : r_j[h]);
    r_lim[h] = tree ? Lb : Lb - n + 1 + r_i[h];
    r_tm[h] = (tree && r_j[h] >= 0) ? p.tree_mask[static_cast<int64_t>(r_b[h]) * n + r_i[h]] : 0xffffffffu;
  }

  cp_async_wait<ST>();  // the Q tile (the oldest group) has landed
  __syncthreads();

  uint32_t qf[D / 16][4];
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks)
    ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3],
                sQ + tile_off<D>((lane & 7) + ((lane >> 3) & 1) * 8, ks * 2 + (lane >> 4)));

  float o[D / 8][4];
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

  for (int jj = 0; jj < nmine; ++jj) {
    // groups so far: Q, the first ST chunks, one per earlier iteration; chunk jj is group jj + 1, so ST - 1 groups
    // may still be pending
    cp_async_wait<ST - 1>();
    __syncwarp();  // everybody's pieces of chunk jj are visible

    const Seg s = segment(jj);
    const uint32_t sK = sRing + (jj % ST) * Cfg::SLOT_BYTES, sV = sK + Cfg::TILE_BYTES;
    if (fused && s.key0 + 16 > s.new_begin && (b_first + s.j) * nG / 16 == rt) {
      // rows of this step's block: into the cache, by the unit that holds the branch's first row
      bf16* kc = const_cast<bf16*>(s.k);
      bf16* vc = const_cast<bf16*>(s.v);
#pragma unroll
      for (int i = 0; i < 16 * CH / 32; ++i) {
        const int idx = lane + i * 32;
        const int row = idx / CH, c = idx % CH;
        const int key = s.key0 + row;
        if (key >= s.new_begin && key < s.len) {
          const int64_t off = static_cast<int64_t>(key) * s.stride + c * 8;
          *reinterpret_cast<uint4*>(kc + off) = lds128(sK + tile_off<D>(row, c));
          *reinterpret_cast<uint4*>(vc + off) = lds128(sV + tile_off<D>(row, c));
        }
      }
    }

    // S (16 rows x 16 keys) = Q K^T
    float sc[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4(b0, b1, b2, b3, sK + tile_off<D>((lane & 7) + (lane >> 4) * 8, ks * 2 + ((lane >> 3) & 1)));
      mma_bf16_16816(sc[0], qf[ks], b0, b1);
      mma_bf16_16816(sc[1], qf[ks], b2, b3);
    }

    // visibility: a prefix key is seen by every valid row, a suffix key by the rows of its branch
    // below their limit (inside the draft block the row's bit mask decides when there is one)
    int lim[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) lim[h] = s.j < 0 ? (r_j[h] >= 0 ? P : 0) : (r_j[h] == s.j ? min(r_lim[h], s.len) : 0);
    const int hist = (tree && s.j >= 0) ? s.len - n : 0x7fffffff;
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int key = s.key0 + nt * 8 + tq * 2 + e;
        const bool in_block = key >= hist;
        const uint32_t bit = 1u << ((key - hist) & 31);
        const bool va = key < lim[0] && (!in_block || (r_tm[0] & bit));
        const bool vb = key < lim[1] && (!in_block || (r_tm[1] & bit));
        sc[nt][e] = va ? sc[nt][e] * p.scale_log2 : -INFINITY;
        sc[nt][2 + e] = vb ? sc[nt][2 + e] * p.scale_log2 : -INFINITY;
        mx[0] = fmaxf(mx[0], sc[nt][e]);
        mx[1] = fmaxf(mx[1], sc[nt][2 + e]);
      }
    float sub[2], al[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(FULL, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(FULL, mx[h], 2));
      const float mn = fmaxf(m_run[h], mx[h]);
      sub[h] = mn == -INFINITY ? 0.f : mn;
      al[h] = fast_exp2(m_run[h] - sub[h]);
      m_run[h] = mn;
      l_run[h] *= al[h];
    }
    if (__any_sync(FULL, al[0] != 1.f || al[1] != 1.f)) {
#pragma unroll
      for (int i = 0; i < D / 8; ++i) {
        o[i][0] *= al[0];
        o[i][1] *= al[0];
        o[i][2] *= al[1];
        o[i][3] *= al[1];
      }
    }
    uint32_t pf[4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const float p0 = fast_exp2(sc[nt][0] - sub[0]), p1 = fast_exp2(sc[nt][1] - sub[0]);
      const float p2 = fast_exp2(sc[nt][2] - sub[1]), p3 = fast_exp2(sc[nt][3] - sub[1]);
      l_run[0] += p0 + p1;
      l_run[1] += p2 + p3;
      pf[nt * 2 + 0] = pack_bf16(p0, p1);
      pf[nt * 2 + 1] = pack_bf16(p2, p3);
    }

    // O += P V over the chunk's 16 keys
#pragma unroll
    for (int dp = 0; dp < D / 16; ++dp) {
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4_trans(b0, b1, b2, b3, sV + tile_off<D>((lane & 7) + ((lane >> 3) & 1) * 8, dp * 2 + (lane >> 4)));
      mma_bf16_16816(o[2 * dp], pf, b0, b1);
      mma_bf16_16816(o[2 * dp + 1], pf, b2, b3);
    }
    __syncwarp();  // the slot is free
    if (jj + ST < nmine) load_chunk(jj + ST);
    cp_async_commit();
  }
  cp_async_wait<0>();
  __syncwarp();  // every lane is done with the ring: it now takes the warp's partial
  pdl_launch_dependents();

  {  // the warp's partial: per row D floats of O, then (m, l)
    float* wO = reinterpret_cast<float*>(smem + (sRing - sQ));
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float l = l_run[h];
      l += __shfl_xor_sync(FULL, l, 1);
      l += __shfl_xor_sync(FULL, l, 2);
      float* dst = wO + (g + h * 8) * Cfg::OSTRIDE;
#pragma unroll
      for (int i = 0; i < D / 8; ++i)
        *reinterpret_cast<float2*>(dst + i * 8 + tq * 2) = make_float2(o[i][2 * h], o[i][2 * h + 1]);
      if (tq == 0) *reinterpret_cast<float2*>(dst + D) = make_float2(m_run[h], l);
    }
  }
  __syncthreads();
  asm volatile("barrier.cluster.wait.aligned;\n" ::: "memory");  // (arrived at the top) every peer is running

  // ---- the warps' states of each row -> the CTA's partial (unnormalised), pushed to the row's owner:
  // row t lives in CTA t % csize, at [t / csize][source rank]
  {
    const unsigned char* rings = smem + (sRing0 - sQ);
    for (int idx = tid; idx < nvalid * (D / 4); idx += Cfg::THREADS) {
      const int row = idx / (D / 4), c4 = idx % (D / 4);
      float mw[NW], lw[NW], M = -INFINITY;
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float2 ml =
            *reinterpret_cast<const float2*>(rings + w * Cfg::RING_BYTES + (row * Cfg::OSTRIDE + D) * 4);
        mw[w] = ml.x;
        lw[w] = ml.y;
        M = fmaxf(M, ml.x);
      }
      float L = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const float wgt = mw[w] == -INFINITY ? 0.f : fast_exp2(mw[w] - M);
        L += lw[w] * wgt;
        const float4 v = *reinterpret_cast<const float4*>(rings + w * Cfg::RING_BYTES +
                                                          (row * Cfg::OSTRIDE + c4 * 4) * 4);
        acc.x += v.x * wgt;
        acc.y += v.y * wgt;
        acc.z += v.z * wgt;
        acc.w += v.w * wgt;
      }
      const uint32_t dst =
          cluster_map(sRecv + ((((row >> clg) << clg) + rank) * Cfg::OSTRIDE) * 4, static_cast<uint32_t>(row & (csize - 1)));
      st_cluster_f4(dst + c4 * 16, acc);
      if (c4 == 0) st_cluster_f2(dst + D * 4, make_float2(M, L));
    }
  }
  cluster_sync_all();  // every CTA's partials have arrived at their owners

  // ---- the cluster's partials of each owned row, in rank order -> output
  constexpr int V = D / 32;
  const float* recv = reinterpret_cast<const float*>(smem + Cfg::Q_BYTES);
  for (int t = rank + csize * warp; t < nvalid; t += csize * NW) {
    const float* mine = recv + ((t >> clg) << clg) * Cfg::OSTRIDE;
    float2 ml = make_float2(-INFINITY, 0.f);
    if (lane < csize) ml = *reinterpret_cast<const float2*>(mine + lane * Cfg::OSTRIDE + D);
    float M = ml.x;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(FULL, M, off));
    const float w_mine = ml.x == -INFINITY ? 0.f : fast_exp2(ml.x - M);
    float Lsum = ml.y * w_mine;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) Lsum += __shfl_xor_sync(FULL, Lsum, off);
    float acc[V];
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] = 0.f;
    for (int c = 0; c < csize; ++c) {
      const float w = __shfl_sync(FULL, w_mine, c);
      const float* src = mine + c * Cfg::OSTRIDE + lane * V;
#pragma unroll
      for (int j = 0; j < V; ++j) acc[j] += src[j] * w;
    }
    const int R = R0 + t;
    const int gg = R % G, tt = R / G, b = tt / n, i = tt % n, h = hk * G + gg;
    const float inv = 1.f / Lsum;
    float* dst = p.out + ((static_cast<int64_t>(b) * n + i) * p.q_heads + h) * D + lane * V;
    if constexpr (V == 4)
      *reinterpret_cast<float4*>(dst) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
    else
      *reinterpret_cast<float2*>(dst) = make_float2(acc[0] * inv, acc[1] * inv);
    if (p.lse && lane == 0)
      p.lse[(static_cast<int64_t>(b) * p.q_heads + h) * n + i] = (M + log2f(Lsum)) * 0.69314718055994530942f;
  }
  // nothing touches a peer's shared memory after the barrier above, so CTAs may leave independently
}

template <int D, int NW, int ST>
static cudaError_t launch_stream_d(const StreamParams& p, const StreamLayers& layers, int units, cudaStream_t st,
                                   LaunchInfo& li) {
  using Cfg = StreamCfg<D, NW, ST>;
  static PerDeviceOnce attr_done;
  if (!attr_done.done()) {
    cudaError_t e = cudaFuncSetAttribute(branch_stream_kernel<D, NW, ST>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         Cfg::SMEM_BYTES);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(branch_stream_kernel<D, NW, ST>, cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  li.launches += 1;
  return launch_pdl_cluster(branch_stream_kernel<D, NW, ST>,
                            dim3(static_cast<unsigned>(units * p.cluster), static_cast<unsigned>(layers.n > 0 ? layers.n : 1)),
                            dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, static_cast<unsigned>(p.cluster), p, layers);
}

bool branch_stream_preferred(int n_branches, int q_heads, int kv_heads, int q_len, int sm_count) {
  // One 16-row tile per kv head: the prefix is fetched once for all branches.  With more rows every tile walks the
  // prefix again (from L2 after the first), which still wins while all units run at once; beyond that the split-KV
  // kernel with 32-row tiles takes over.
  const int64_t tiles = (static_cast<int64_t>(n_branches) * q_len * (q_heads / kv_heads) + 15) / 16;
  return tiles == 1 || tiles * kv_heads <= sm_count;
}

static cudaError_t launch_stream(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                                 const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len,
                                 int n_branches, int q_heads, int q_len, float scale, float* out, float* lse,
                                 cudaStream_t st, LaunchInfo& li, const bf16* k_new, const bf16* v_new,
                                 const StreamLayers& layers) {
  StreamParams p;
  p.q = q;
  p.prefix = prefix;
  p.suffix = suffix;
  p.d_suffix_len = d_suffix_len;
  p.tree_mask = d_tree_mask;
  p.k_new = k_new;
  p.v_new = v_new;
  p.prefix_len = prefix_len;
  p.max_suffix_len = max_suffix_len;
  p.n_branches = n_branches;
  p.q_heads = q_heads;
  p.group = q_heads / suffix.kv_heads;
  p.q_len = q_len;
  const int rows = n_branches * q_len * p.group;
  p.row_tiles = (rows + 15) / 16;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.out = out;
  p.lse = lse;
  const int units = suffix.kv_heads * p.row_tiles;
  // the largest portable cluster that keeps every CTA (of one problem) resident at once
  int c = 1;
  while (c < 8 && units * c * 2 <= li.sm_count * kStreamCtasPerSm) c *= 2;
  // no more CTAs than 16-key chunks of work per unit warrant
  const int64_t chunks = (prefix_len + 15) / 16 + static_cast<int64_t>(max_suffix_len + 15) / 16;
  while (c > 1 && chunks < static_cast<int64_t>(c) * 8) c /= 2;
  p.cluster = c;
  p.cluster_log2 = c == 8 ? 3 : (c == 4 ? 2 : (c == 2 ? 1 : 0));
  if (suffix.head_dim == 128) return launch_stream_d<128, kStreamWarps, kStreamStages>(p, layers, units, st, li);
  return launch_stream_d<64, kStreamWarps, kStreamStages>(p, layers, units, st, li);
}

cudaError_t launch_branch_stream(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                                 const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len,
                                 int n_branches, int q_heads, int q_len, float scale, float* out, float* lse,
                                 cudaStream_t st, LaunchInfo& li, const bf16* k_new, const bf16* v_new) {
  StreamLayers none;
  none.n = 0;
  return launch_stream(q, prefix, prefix_len, suffix, d_suffix_len, d_tree_mask, max_suffix_len, n_branches, q_heads,
                       q_len, scale, out, lse, st, li, k_new, v_new, none);
}

cudaError_t launch_branch_stream_layers(const BranchLayerTensors* layers, int n_layers, const CacheView& prefix,
                                        int prefix_len, const CacheView& suffix, const int32_t* d_suffix_len,
                                        int max_suffix_len, int n_branches, int q_heads, int q_len, float scale,
                                        cudaStream_t st, LaunchInfo& li) {
  for (int first = 0; first < n_layers; first += kBranchMaxLayersPerLaunch) {
    StreamLayers batch;
    batch.n = std::min(kBranchMaxLayersPerLaunch, n_layers - first);
    for (int i = 0; i < batch.n; ++i) {
      const BranchLayerTensors& t = layers[first + i];
      batch.l[i] = StreamLayerPtrs{t.q, t.k_new, t.v_new, t.pk, t.pv, t.sk, t.sv, t.out, t.lse};
    }
    const BranchLayerTensors& t0 = layers[first];
    cudaError_t e = launch_stream(t0.q, prefix, prefix_len, suffix, d_suffix_len, nullptr, max_suffix_len, n_branches,
                                  q_heads, q_len, scale, t0.out, t0.lse, st, li, t0.k_new, t0.v_new, batch);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace jup
