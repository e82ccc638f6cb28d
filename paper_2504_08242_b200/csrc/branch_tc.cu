// Branch attention with many stacked query rows per kv head on the 5th-generation tensor cores (paper Sec. V-A,
// Fig. 7 step 3: the k draft tokens of every request are verified in one pass; Sec. V-B, Fig. 8: all
// point-extending requests share the prompt's KVCache).
//
// head_dim 128.  The stacked rows of a kv head -- (branch, draft token, head of the group), in that order -- are
// cut into tiles of 128 rows.  A unit = (kv head, row tile).  Every row belongs to one branch and may see the shared
// prefix plus that branch's suffix, so a row keeps ONE online-softmax state in its TMEM lane while the unit walks
//     prefix | suffix of the tile's first branch | ... | suffix of its last branch
// in tiles of 128 keys: a prefix tile is visible to every row, a suffix tile to the rows of its branch below
// their causal limit (or tree mask).  A prefix K/V tile is therefore fetched once per 128 rows, not once per branch.
//
// `ctas_per_unit` CTAs share a unit: the prefix tiles are cut into equal contiguous ranges, one per CTA, and so
// are the suffix tiles (the prefix share does not depend on the device-side lengths, so its first loads are in
// flight while the lengths arrive).  Inside a CTA:
//   loader warp  : TMA (tiled, 128-byte swizzle) Q once -- one box [128/G tokens][G heads][64] lands in stacked-row
//                  order -- then the K/V tiles of the CTA's list into 3-stage rings
//   patch warp   : the last tiles of a branch's suffix hold rows that TMA cannot know about: rows at or beyond the
//                  device-side length (dead; their V rows are zeroed so that 0 x NaN never reaches an accumulator)
//                  and, with the fused KVCache write, the rows of this step's block, which are read from
//                  k_new / v_new into the tile (and stored into the cache by the unit that owns the branch)
//   MMA warp     : one thread issues tcgen05.mma  S = Q K^T  and  O += P V, accumulators in TMEM
//   softmax WGs  : two warpgroups run two independent online-softmax streams over the even and the odd tiles of
//                  the CTA's list (one thread per row); a warp none of whose rows sees a tile only zeroes its P
// TMEM (512 columns): S_0 | S_1 | O_0 | O_1.
// At the end the two streams are merged.  With one CTA per unit the result is normalised and written with tiled
// stores.  Otherwise the CTA writes its unnormalised partial (O, m, l) to scratch and takes a ticket on the
// unit's counter; the CTA that takes the last ticket merges the unit's partials in CTA order (so the result
// never depends on timing), puts the counter back to zero and writes the output.  Nothing waits on another CTA.
// All mbarrier waits are bounded; on expiry the CTA sets the status word, drains its own copies and MMAs,
// frees TMEM and returns.
#include <algorithm>

#include "host_checks.h"
#include "kernels.h"
#include "tc_common.cuh"
#include "tc_softmax.cuh"
#include "tmap.h"

namespace jup {

constexpr int BT_D = 128;
constexpr int BT_BM = 128;             // stacked rows per tile
constexpr int BT_BN = 128;             // keys per KV tile
constexpr int BT_TILE_BYTES = 32768;   // 128 x 128 bf16
constexpr int BT_PANEL_BYTES = 16384;  // 128 rows x 64 elements
constexpr int BT_KV_STAGES = 3;
constexpr int BT_MAX_TILES = 160;      // tiles one CTA can list
constexpr int BT_MAX_BRANCHES = 32;    // branches with a row in one 128-row tile
constexpr int BT_MAX_CTAS = 16;        // CTAs per unit
constexpr int BT_BOX_FLOATS = BT_BM * 32;
constexpr int BT_PART_FLOATS = BT_BM * BT_D;  // one CTA's partial accumulator
constexpr int BT_ML_FLOATS = BT_BM * 2;       // and its (m, l) pairs

struct BtParams {
  int n_branches, q_len, q_heads, group, kv_heads;
  int prefix_len, max_suffix_len;
  int row_tiles;      // 128-row tiles per kv head
  int ctas_per_unit;
  float scale_log2;
  long long wait_limit;
  const int32_t* d_suffix_len;
  const uint32_t* tree_mask;  // nullable: [n_branches][q_len] ancestor bit masks of the draft block
  const bf16* k_new;          // nullable: fused KVCache write, [n_branches][q_len][kv_heads][128]
  const bf16* v_new;
  bf16* k_cache;              // the suffix cache (written only with the fused write)
  bf16* v_cache;
  int64_t sb, sh, sr;
  float* lse;
  int* status;
  int* counters;  // [units], zero on entry and on exit
  float* part;    // [units][ctas_per_unit][32 column chunks][128 rows] float4
  float* ml;      // [units][ctas_per_unit][128 rows] (m, l)
};

// shared memory: [Q][K ring][V ring][barriers, flags][lengths][tile table]
constexpr int BT_SMEM_Q = 0;
constexpr int BT_SMEM_K = BT_TILE_BYTES;
constexpr int BT_SMEM_V = BT_SMEM_K + BT_KV_STAGES * BT_TILE_BYTES;
constexpr int BT_SMEM_BAR = BT_SMEM_V + BT_KV_STAGES * BT_TILE_BYTES;
constexpr int BT_SMEM_LEN = BT_SMEM_BAR + 256;
constexpr int BT_SMEM_TABLE = BT_SMEM_LEN + 2 * BT_MAX_BRANCHES * 4;
constexpr int BT_SMEM_BYTES = BT_SMEM_TABLE + BT_MAX_TILES * 4 + 1024;  // + slack for 1024-byte alignment
static_assert(BT_SMEM_BYTES <= 227 * 1024, "shared memory per CTA");
constexpr int BT_LOADER_WARP = 8,  // warps 0..7: the two softmax warpgroups
               BT_MMA_WARP = 9, BT_PATCH_WARP = 10;
constexpr int BT_THREADS = 32 * 11;

enum {
  BT_Q_FULL = 0,
  BT_K_FULL = 1,    // [3]
  BT_K_EMPTY = 4,   // [3]
  BT_V_FULL = 7,    // [3]
  BT_V_EMPTY = 10,  // [3]
  BT_PATCHED = 13,  // [3] the patch warp is done with the slot's tile
  BT_S_FULL = 16,   // [2]
  BT_P_FULL = 18,   // [2]
  BT_O_READY = 20,  // [2]
  BT_DRAIN = 22,
  BT_BAR_COUNT = 23
};

// tile table entry: bits [0,8) branch as an index into the tile's branches (0xff: shared prefix),
// [8,24) tile number inside the segment, bit 24: the patch warp has work on it
__device__ __forceinline__ int bt_seg(uint32_t e) { return static_cast<int>(e & 0xffu); }
__device__ __forceinline__ int bt_tile(uint32_t e) { return static_cast<int>((e >> 8) & 0xffffu); }
__device__ __forceinline__ bool bt_patch(uint32_t e) { return (e >> 24) & 1u; }

__global__ void __launch_bounds__(BT_THREADS, 1)
branch_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_pk,
                 const __grid_constant__ CUtensorMap tm_pv, const __grid_constant__ CUtensorMap tm_sk,
                 const __grid_constant__ CUtensorMap tm_sv, const __grid_constant__ CUtensorMap tm_o, BtParams p) {
  constexpr int KV_STAGES = BT_KV_STAGES;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base + BT_SMEM_Q, sK = smem_base + BT_SMEM_K, sV = smem_base + BT_SMEM_V;
  const uint32_t sBar = smem_base + BT_SMEM_BAR;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + BT_SMEM_BAR + 8 * BT_BAR_COUNT);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + BT_SMEM_BAR + 8 * BT_BAR_COUNT + 8);
  volatile int* n_tiles_slot = reinterpret_cast<volatile int*>(smem_gen + BT_SMEM_BAR + 8 * BT_BAR_COUNT + 16);
  volatile int* last_slot = reinterpret_cast<volatile int*>(smem_gen + BT_SMEM_BAR + 8 * BT_BAR_COUNT + 24);
  int* len_s = reinterpret_cast<int*>(smem_gen + BT_SMEM_LEN);  // clamped suffix length of the tile's branches
  int* cum_s = len_s + BT_MAX_BRANCHES;                         // one past the last suffix tile of each
  uint32_t* table = reinterpret_cast<uint32_t*>(smem_gen + BT_SMEM_TABLE);
  auto bar = [&](int i) { return sBar + 8u * i; };
  const long long wl = p.wait_limit;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int C = p.ctas_per_unit;
  const int unit = blockIdx.x / C, crank = blockIdx.x % C;
  const int rt = unit % p.row_tiles, hk = unit / p.row_tiles;
  const int n = p.q_len, G = p.group, nG = n * G;
  const int rows_total = p.n_branches * nG;
  const int R0 = rt * BT_BM;
  const int rows_here = min(BT_BM, rows_total - R0);
  const int b_first = R0 / nG;
  const int nb = (R0 + rows_here - 1) / nG - b_first + 1;  // branches with a row in this tile
  const int P = p.prefix_len;
  const bool fused = p.k_new != nullptr;
  // this CTA's share of the prefix tiles: known without any memory access
  const int Tp = (P + BT_BN - 1) / BT_BN;
  const int p0 = Tp * crank / C, npre = Tp * (crank + 1) / C - p0;

  // ---- set-up
  if (threadIdx.x == 0) {
    for (int i = 0; i < BT_BAR_COUNT; ++i) mbar_init(bar(i), (i == BT_P_FULL || i == BT_P_FULL + 1) ? 128u : 1u);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == BT_MMA_WARP) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish();
  } else if (warp == BT_LOADER_WARP && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_sk);
    tma_prefetch_desc(&tm_sv);
    if (Tp > 0) {
      tma_prefetch_desc(&tm_pk);
      tma_prefetch_desc(&tm_pv);
    }
    tma_prefetch_desc(&tm_o);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();  // everything above overlapped the previous kernel's tail; global memory is touched from here on

  auto load_tile = [&](int s, uint32_t e) {  // K and V of list entry e into the ring slot of sequence number s
    const int slot = s % KV_STAGES;
    const bool pre = bt_seg(e) == 0xff;
    const int row = bt_tile(e) * BT_BN, bb = pre ? 0 : b_first + bt_seg(e);
    mbar_expect_tx(bar(BT_K_FULL + slot), BT_TILE_BYTES);
    const CUtensorMap* mk = pre ? &tm_pk : &tm_sk;
    tma_load_4d(sK + slot * BT_TILE_BYTES, mk, bar(BT_K_FULL + slot), 0, row, hk, bb);
    tma_load_4d(sK + slot * BT_TILE_BYTES + BT_PANEL_BYTES, mk, bar(BT_K_FULL + slot), 64, row, hk, bb);
    mbar_expect_tx(bar(BT_V_FULL + slot), BT_TILE_BYTES);
    const CUtensorMap* mv = pre ? &tm_pv : &tm_sv;
    tma_load_4d(sV + slot * BT_TILE_BYTES, mv, bar(BT_V_FULL + slot), 0, row, hk, bb);
    tma_load_4d(sV + slot * BT_TILE_BYTES + BT_PANEL_BYTES, mv, bar(BT_V_FULL + slot), 64, row, hk, bb);
  };
  const int pre_issued = min(npre, KV_STAGES);
  if (warp == BT_LOADER_WARP && lane == 0) {
    // Q: token rows R0 / G .. of heads hk G .., one box per 64-column panel
    mbar_expect_tx(bar(BT_Q_FULL), BT_TILE_BYTES);
    tma_load_4d(sQ, &tm_q, bar(BT_Q_FULL), 0, hk * G, R0 / G, 0);
    tma_load_4d(sQ + BT_PANEL_BYTES, &tm_q, bar(BT_Q_FULL), 64, hk * G, R0 / G, 0);
    for (int s = 0; s < pre_issued; ++s) load_tile(s, 0xffu | (static_cast<uint32_t>(p0 + s) << 8));
  } else if (warp == 0) {
    // ---- tile list of this CTA: its prefix share, then its share of the suffix tiles of the tile's branches
    int L = 0;
    if (lane < nb) {
      L = __ldg(p.d_suffix_len + b_first + lane);
      L = L < n ? n : (L > p.max_suffix_len ? p.max_suffix_len : L);
    }
    int cum = (L + BT_BN - 1) / BT_BN;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, cum, o);
      if (lane >= o) cum += t;
    }
    len_s[lane] = L;
    cum_s[lane] = cum;
    const int Ts = __shfl_sync(0xffffffffu, cum, 31);
    const int s0 = static_cast<int>(static_cast<int64_t>(Ts) * crank / C);
    const int nsuf = static_cast<int>(static_cast<int64_t>(Ts) * (crank + 1) / C) - s0;
    __syncwarp();
    const int total = min(npre + nsuf, BT_MAX_TILES);  // the host sized the launch so that the list fits
    for (int u = lane; u < total; u += 32) {
      uint32_t e;
      if (u < npre) {
        e = 0xffu | (static_cast<uint32_t>(p0 + u) << 8);
      } else {
        const int g = s0 + u - npre;
        int j = 0;
        while (j < nb - 1 && cum_s[j] <= g) ++j;
        const int tile = g - (j > 0 ? cum_s[j - 1] : 0);
        const int first_special = fused ? len_s[j] - n : len_s[j];  // first row that is new or dead
        const bool patch = (tile + 1) * BT_BN > first_special;
        e = static_cast<uint32_t>(j) | (static_cast<uint32_t>(tile) << 8) | (patch ? 1u << 24 : 0u);
      }
      table[u] = e;
    }
    if (lane == 0) *n_tiles_slot = total;
  }
  __syncthreads();
  const int Tall = *n_tiles_slot;
  const int T[2] = {(Tall + 1) >> 1, Tall >> 1};  // stream x takes the sequence numbers 2 i + x

  if (warp == BT_LOADER_WARP) {
    // =============================================================== loader
    if (lane == 0) {
      bool ok = true;
      int issued = pre_issued;
      for (int s = pre_issued; s < Tall && ok; ++s) {
        const int slot = s % KV_STAGES, u = s / KV_STAGES;
        if (u > 0) {
          ok = mbar_wait(bar(BT_K_EMPTY + slot), (u - 1) & 1, abort_flag, p.status, wl) &&
               mbar_wait(bar(BT_V_EMPTY + slot), (u - 1) & 1, abort_flag, p.status, wl);
          if (!ok) break;
        }
        load_tile(s, table[s]);
        issued = s + 1;
      }
      if (*abort_flag) {
        // wait (bounded) until every copy this thread started has landed before shared memory is released
        int dummy = 0;
        volatile int* none = &dummy;
        for (int s = max(0, issued - KV_STAGES); s < issued; ++s) {
          mbar_wait(bar(BT_K_FULL + s % KV_STAGES), (s / KV_STAGES) & 1, none, nullptr, wl);
          mbar_wait(bar(BT_V_FULL + s % KV_STAGES), (s / KV_STAGES) & 1, none, nullptr, wl);
        }
        mbar_wait(bar(BT_Q_FULL), 0, none, nullptr, wl);
      }
    }
    __syncwarp();
  } else if (warp == BT_PATCH_WARP) {
    // =============================================================== patch warp
    bool ok = true;
    for (int s = 0; s < Tall && ok; ++s) {
      const int slot = s % KV_STAGES, u = s / KV_STAGES;
      ok = mbar_wait(bar(BT_K_FULL + slot), u & 1, abort_flag, p.status, wl) &&
           mbar_wait(bar(BT_V_FULL + slot), u & 1, abort_flag, p.status, wl);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint32_t e = table[s];
      if (bt_patch(e)) {
        const int j = bt_seg(e), b = b_first + j, L = len_s[j], key0 = bt_tile(e) * BT_BN;
        const int new_begin = fused ? L - n : L;
        const int r_begin = max(new_begin - key0, 0);
        // the unit that holds the branch's first stacked row stores the block into the cache
        const bool writer = fused && (b * nG) / BT_BM == rt;
        const uint32_t kslot = sK + slot * BT_TILE_BYTES, vslot = sV + slot * BT_TILE_BYTES;
        for (int idx = lane; idx < (BT_BN - r_begin) * 16; idx += 32) {
          const int r = r_begin + (idx >> 4), c = idx & 15;
          const int key = key0 + r;
          // 16-byte piece c of row r in the 128-byte-swizzled two-panel tile
          const uint32_t off = (c >> 3) * BT_PANEL_BYTES + r * 128 + (((c & 7) ^ (r & 7)) << 4);
          if (key < L) {  // a row of this step's block
            const int64_t src = ((static_cast<int64_t>(b) * n + (key - new_begin)) * p.kv_heads + hk) * BT_D + c * 8;
            const uint4 kk = __ldg(reinterpret_cast<const uint4*>(p.k_new + src));
            const uint4 vv = __ldg(reinterpret_cast<const uint4*>(p.v_new + src));
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};\n" ::"r"(kslot + off), "r"(kk.x), "r"(kk.y), "r"(kk.z),
                         "r"(kk.w)
                         : "memory");
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};\n" ::"r"(vslot + off), "r"(vv.x), "r"(vv.y), "r"(vv.z),
                         "r"(vv.w)
                         : "memory");
            if (writer) {
              const int64_t dst = b * p.sb + hk * p.sh + static_cast<int64_t>(key) * p.sr + c * 8;
              *reinterpret_cast<uint4*>(p.k_cache + dst) = kk;
              *reinterpret_cast<uint4*>(p.v_cache + dst) = vv;
            }
          } else {  // a dead row: its scores are masked, its V row must not poison the accumulator
            asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};\n" ::"r"(vslot + off), "r"(0u) : "memory");
          }
        }
        fence_proxy_async();  // the tensor cores read the slot through the async proxy
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(BT_PATCHED + slot));
    }
  } else if (warp == BT_MMA_WARP) {
    // =============================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = tc_idesc_bf16(BT_BM, BT_BN, false, false);
      constexpr uint32_t idesc_pv = tc_idesc_bf16(BT_BM, BT_D, false, true);
      auto s_col = [&](int x) { return tmem + x * 128; };
      auto o_col = [&](int x) { return tmem + 256 + x * 128; };
      auto issue_qk = [&](int x, int s) {  // S(x) = Q K^T, K of sequence number s
        const uint32_t kb = sK + (s % KV_STAGES) * BT_TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < BT_D / 16; ++ks) {
          const uint32_t off = (ks >> 2) * BT_PANEL_BYTES + (ks & 3) * 32;
          tc_mma_ss(s_col(x), tc_smem_desc(sQ + off, 16, 1024), tc_smem_desc(kb + off, 16, 1024), idesc_qk, ks > 0);
        }
      };
      auto issue_pv = [&](int x, int s, bool first) {  // O(x) (+)= P(x) V, V of sequence number s
        const uint32_t vb = sV + (s % KV_STAGES) * BT_TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < BT_BN / 16; ++ks)
          tc_mma_ts(o_col(x), s_col(x) + ks * 8, tc_smem_desc(vb + ks * 2048, BT_PANEL_BYTES, 1024), idesc_pv,
                    (!first || ks > 0));
      };
      bool ok = true;
      int ready = -1;  // tiles up to this sequence number have landed and are patched
      auto need = [&](int s) {
        while (ready < s && ok) {
          ++ready;
          const int slot = ready % KV_STAGES, u = ready / KV_STAGES;
          ok = mbar_wait(bar(BT_K_FULL + slot), u & 1, abort_flag, p.status, wl) &&
               mbar_wait(bar(BT_V_FULL + slot), u & 1, abort_flag, p.status, wl) &&
               mbar_wait(bar(BT_PATCHED + slot), u & 1, abort_flag, p.status, wl);
          tc_fence_after();
        }
      };
      ok = mbar_wait(bar(BT_Q_FULL), 0, abort_flag, p.status, wl);  // (also when the list is empty: the copy must land)
#pragma unroll
      for (int x = 0; x < 2; ++x) {  // prologue: S(x) of the stream's first tile
        if (T[x] == 0 || !ok) continue;
        need(x);
        if (!ok) break;
        issue_qk(x, x);
        tc_commit(bar(BT_S_FULL + x));
        tc_commit(bar(BT_K_EMPTY + x % KV_STAGES));
      }
      for (int j = 0; j < T[0] && ok; ++j) {
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          if (j >= T[x] || !ok) continue;
          const int s = 2 * j + x, sn = s + 2;
          need(s);
          ok = ok && mbar_wait(bar(BT_P_FULL + x), j & 1, abort_flag, p.status, wl);
          if (!ok) break;
          tc_fence_after();
          issue_pv(x, s, j == 0);
          tc_commit(bar(BT_O_READY + x));
          tc_commit(bar(BT_V_EMPTY + s % KV_STAGES));
          if (j + 1 < T[x]) {
            need(sn);
            if (!ok) break;
            issue_qk(x, sn);
            tc_commit(bar(BT_S_FULL + x));
            tc_commit(bar(BT_K_EMPTY + sn % KV_STAGES));
          }
        }
      }
      if (!ok) {  // make sure no MMA of this thread is still running before TMEM and smem go away
        int dummy = 0;
        tc_commit(bar(BT_DRAIN));
        mbar_wait(bar(BT_DRAIN), 0, &dummy, nullptr, wl);
      }
    }
    __syncwarp();
  } else {
    // =============================================================== softmax warpgroups (streams)
    const int x = warp >> 2;
    const int row_in_tile = (warp & 3) * 32 + lane;
    const int R = R0 + row_in_tile;
    const bool row_valid = R < rows_total;
    const int tok = R / G, hq = hk * G + R % G;       // token (branch, draft row) and query head of this row
    const int rb = tok / n, ri = tok % n;
    const int rj = row_valid ? rb - b_first : -1;    // the row's branch as an index into the tile's branches
    // draft rows of the block this row may see, as bits: its ancestors and itself (a chain: rows 0..i)
    const uint32_t tm = !row_valid ? 0u
                        : (p.tree_mask ? __ldg(p.tree_mask + static_cast<int64_t>(rb) * n + ri) : (2u << ri) - 1u) &
                              ((n < 32 ? (1u << n) : 0u) - 1u);
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + x * 128;
    const uint32_t tO = tmem + lane_base + 256 + x * 128;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    const int Tx = T[x];
    for (int j = 0; j < Tx && ok; ++j) {
      ok = mbar_wait(bar(BT_S_FULL + x), j & 1, abort_flag, p.status, wl);
      if (!ok) break;
      tc_fence_after();
      // ---- which columns of the tile this row sees
      const uint32_t e = table[2 * j + x];
      const int key0 = bt_tile(e) * BT_BN;
      ColumnBits allow;
      bool full, any;
      if (bt_seg(e) == 0xff) {  // shared prefix: every row, up to its end
        const int cnt = P - key0;
        full = cnt >= BT_BN;
        any = true;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int k = cnt - 32 * w;
          allow.w[w] = k >= 32 ? 0xffffffffu : (k <= 0 ? 0u : (1u << k) - 1u);
        }
      } else if (bt_seg(e) == rj) {  // the row's own branch: rows before the block, then the block by the mask
        const int hist = len_s[rj] - n - key0;  // column of the block's first row
        full = hist >= BT_BN;
        any = hist > 0 || tm != 0u;  // (hist + n > 0 always holds for a listed tile)
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int k = hist - 32 * w;
          const uint32_t before = k >= 32 ? 0xffffffffu : (k <= 0 ? 0u : (1u << k) - 1u);
          const uint32_t block = k >= 32 ? 0u : (k >= 0 ? tm << k : (k > -32 ? tm >> (-k) : 0u));
          allow.w[w] = before | block;
        }
        any = (allow.w[0] | allow.w[1] | allow.w[2] | allow.w[3]) != 0u;
      } else {  // another branch's suffix
        full = false;
        any = false;
        allow.w[0] = allow.w[1] = allow.w[2] = allow.w[3] = 0u;
      }
      auto wait_o = [&] { return mbar_wait(bar(BT_O_READY + x), (j - 1) & 1, abort_flag, p.status, wl); };
      if (__any_sync(0xffffffffu, any)) {
        const bool masked = !__all_sync(0xffffffffu, full);
        ok = softmax_tile_step<true>(tS, tO, j, masked, allow, c, m_ref, l, wait_o);
      } else {  // no row of this warp sees the tile: P = 0, nothing else changes
        uint32_t z[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) z[i] = 0u;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) tmem_st16(tS + q4 * 16, z);
        tc_wait_st();
        if (j > 0) ok = wait_o();
      }
      if (!ok) break;
      tc_fence_before();
      mbar_arrive(bar(BT_P_FULL + x));
    }
    pdl_launch_dependents();  // the next kernel of the stream may start its own set-up now

    // ---- merge of the two streams.  Every softmax thread reaches the named barriers below, even one that gave up on
    // a wait (it only skips its global stores).  (m, l) of a row cross through shared memory -- the K slot of the
    // stream's last tile, free once its accumulator is complete; a stream without tiles owns slot x, never filled or
    // long free -- the accumulators are read straight from TMEM: this warpgroup combines columns [64 x, 64 x + 64).
    auto ml_of = [&](int y) {
      const int slot = T[y] > 0 ? (2 * (T[y] - 1) + y) % KV_STAGES : y;
      return reinterpret_cast<float2*>(smem_gen + BT_SMEM_K + slot * BT_TILE_BYTES);
    };
    if (Tx > 0) ok = mbar_wait(bar(BT_O_READY + x), (Tx - 1) & 1, abort_flag, p.status, wl) && ok;
    ml_of(x)[row_in_tile] = make_float2(m_ref, l);
    tc_fence_before();
    asm volatile("bar.sync 3, 256;\n" ::: "memory");
    tc_fence_after();
    const float2 oth = ml_of(1 - x)[row_in_tile];
    // a stream whose tiles were all hidden from this row has l = 0 and takes no part
    const float m_own = l > 0.f ? m_ref : -INFINITY, m_oth = oth.y > 0.f ? oth.x : -INFINITY;
    const float m = fmaxf(m_own, m_oth);
    const float w_own = l > 0.f ? fast_exp2(m_own - m) : 0.f, w_oth = oth.y > 0.f ? fast_exp2(m_oth - m) : 0.f;
    const float lsum = l * w_own + oth.y * w_oth;
    const bool has_own = Tx > 0, has_oth = T[1 - x] > 0;  // a stream without tiles never wrote its accumulator
    const uint32_t tOwn = tmem + lane_base + 256 + x * 128 + x * 64;
    const uint32_t tOth = tmem + lane_base + 256 + (1 - x) * 128 + x * 64;
    const int tid_t = threadIdx.x & 127;
    // staging for the tiled stores of the output: the Q buffer for warpgroup 0, the first V slot for warpgroup 1
    // (every MMA and copy of the CTA is complete once both streams have seen their last accumulator)
    float* stage = reinterpret_cast<float*>(smem_gen + (x == 0 ? BT_SMEM_Q : BT_SMEM_V));
    const uint32_t stage_addr = smem_base + (x == 0 ? BT_SMEM_Q : BT_SMEM_V);
    auto store_box = [&](int q2, const float (&v)[32], bool write) {  // columns [64 x + 32 q2, + 32) of all 128 rows
      stage_box_row(stage + q2 * BT_BOX_FLOATS, row_in_tile, v);
      fence_proxy_async();
      asm volatile("bar.sync %0, 128;\n" ::"r"(1 + x) : "memory");
      if (tid_t == 0 && write) {
        tma_store_4d(&tm_o, stage_addr + q2 * BT_BOX_FLOATS * 4, x * 64 + q2 * 32, hk * G, R0 / G, 0);
        tma_store_commit();
      }
    };
    auto store_lse = [&](float mm, float ll) {
      if (x == 0 && p.lse && row_valid)
        p.lse[(static_cast<int64_t>(rb) * p.q_heads + hq) * n + ri] = (mm + log2f(ll)) * 0.69314718055994530942f;
    };
    if (C == 1) {
      const float inv = 1.f / lsum;
      const float a_own = w_own * inv, a_oth = w_oth * inv;
#pragma unroll
      for (int q2 = 0; q2 < 2; ++q2) {
        uint32_t o[32], o2[32];
        if (has_own) tmem_ld32(tOwn + q2 * 32, o);
        if (has_oth) tmem_ld32(tOth + q2 * 32, o2);
        tc_wait_ld();
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          v[i] = has_own ? __uint_as_float(o[i]) * a_own : 0.f;
          if (has_oth) v[i] = fmaf(__uint_as_float(o2[i]), a_oth, v[i]);
        }
        store_box(q2, v, ok);
      }
      if (tid_t == 0) tma_store_wait_read();
      if (ok) store_lse(m, lsum);
    } else {
      // ---- this CTA's partial -> scratch: [column chunk][row] float4, so a warp writes 512 contiguous bytes
      float4* gpart = reinterpret_cast<float4*>(p.part + (static_cast<size_t>(unit) * C + crank) * BT_PART_FLOATS);
      float2* gml = reinterpret_cast<float2*>(p.ml + (static_cast<size_t>(unit) * C + crank) * BT_ML_FLOATS);
#pragma unroll
      for (int q2 = 0; q2 < 2; ++q2) {
        uint32_t o[32], o2[32];
        if (has_own) tmem_ld32(tOwn + q2 * 32, o);
        if (has_oth) tmem_ld32(tOth + q2 * 32, o2);
        tc_wait_ld();
#pragma unroll
        for (int cc = 0; cc < 8; ++cc) {
          float v[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            v[i] = has_own ? __uint_as_float(o[4 * cc + i]) * w_own : 0.f;
            if (has_oth) v[i] = fmaf(__uint_as_float(o2[4 * cc + i]), w_oth, v[i]);
          }
          gpart[(x * 16 + q2 * 8 + cc) * BT_BM + row_in_tile] = make_float4(v[0], v[1], v[2], v[3]);
        }
      }
      if (x == 0) gml[row_in_tile] = make_float2(lsum > 0.f ? m : -INFINITY, lsum);
      // ---- ticket: the partial above must be visible before the ticket is
      __threadfence();
      asm volatile("bar.sync 3, 256;\n" ::: "memory");
      if (threadIdx.x == 0) {
        int* cnt = p.counters + unit;
        const bool last = atomicAdd(cnt, 1) == C - 1;
        if (last) *cnt = 0;  // every CTA of the unit has taken its ticket: ready for the next call
        __threadfence();     // the others' partials are read after this
        *last_slot = last ? 1 : 0;
      }
      asm volatile("bar.sync 3, 256;\n" ::: "memory");
      if (*last_slot) {
        // ---- the unit's partials in CTA order -> output
        const bool clean = ok && *reinterpret_cast<volatile int*>(p.status) == 0;  // nobody gave up on a wait
        const float2* uml = reinterpret_cast<const float2*>(p.ml + static_cast<size_t>(unit) * C * BT_ML_FLOATS);
        const float4* upart = reinterpret_cast<const float4*>(p.part + static_cast<size_t>(unit) * C * BT_PART_FLOATS);
        // (weights in registers: the loops over the unit's CTAs are unrolled to their upper bound)
        float wgt[BT_MAX_CTAS], lcr[BT_MAX_CTAS];
        float M = -INFINITY;
#pragma unroll
        for (int cr = 0; cr < BT_MAX_CTAS; ++cr) {
          const float2 v = cr < C ? __ldcg(uml + cr * BT_BM + row_in_tile) : make_float2(-INFINITY, 0.f);
          wgt[cr] = v.y > 0.f ? v.x : -INFINITY;  // a CTA whose tiles were all hidden from the row has l = 0
          lcr[cr] = v.y;
          M = fmaxf(M, wgt[cr]);
        }
        float lall = 0.f;
#pragma unroll
        for (int cr = 0; cr < BT_MAX_CTAS; ++cr) {
          wgt[cr] = wgt[cr] == -INFINITY ? 0.f : fast_exp2(wgt[cr] - M);
          lall = fmaf(wgt[cr], lcr[cr], lall);
        }
        const float inv = 1.f / lall;
#pragma unroll
        for (int q2 = 0; q2 < 2; ++q2) {
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0.f;
#pragma unroll
          for (int cr = 0; cr < BT_MAX_CTAS; ++cr) {
            const float w = wgt[cr];
            if (cr >= C || w == 0.f) continue;  // (also a CTA without tiles, which wrote no accumulator)
            const float4* src = upart + static_cast<size_t>(cr) * (BT_PART_FLOATS / 4) + (x * 16 + q2 * 8) * BT_BM + row_in_tile;
            float4 t[8];
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) t[cc] = __ldcg(src + cc * BT_BM);
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) {
              v[4 * cc] = fmaf(w, t[cc].x, v[4 * cc]);
              v[4 * cc + 1] = fmaf(w, t[cc].y, v[4 * cc + 1]);
              v[4 * cc + 2] = fmaf(w, t[cc].z, v[4 * cc + 2]);
              v[4 * cc + 3] = fmaf(w, t[cc].w, v[4 * cc + 3]);
            }
          }
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] *= inv;
          store_box(q2, v, clean);
        }
        if (tid_t == 0) tma_store_wait_read();
        if (clean) store_lse(M, lall);
      }
    }
  }

  // ---- tear-down
  tc_fence_before();
  __syncthreads();
  if (warp == BT_MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---------------------------------------------------------------- host side

struct BtPlan {
  int row_tiles, units, ctas_per_unit;
  bool ok;
};

static BtPlan bt_plan(int prefix_len, int max_suffix_len, int n_branches, int q_heads, int kv_heads, int q_len,
                      int sm_count) {
  BtPlan pl = {0, 0, 1, false};
  const int G = q_heads / kv_heads, nG = q_len * G;
  if (G > BT_BM || (G & (G - 1)) != 0) return pl;               // a Q box holds whole tokens: G divides 128
  if ((BT_BM - 1) / nG + 2 > BT_MAX_BRANCHES) return pl;        // branches with a row in one tile
  const int64_t rows = static_cast<int64_t>(n_branches) * nG;
  const int64_t row_tiles = (rows + BT_BM - 1) / BT_BM;
  const int64_t units = row_tiles * kv_heads;
  if (units > 65536 / 4) return pl;                              // one counter per unit in the 64 KiB counter block
  const int64_t Tp = (static_cast<int64_t>(prefix_len) + BT_BN - 1) / BT_BN;
  if (Tp > 0xffff) return pl;
  const int nb_max = static_cast<int>(std::min<int64_t>((BT_BM - 1) / nG + 2, n_branches));
  const int64_t Ts_max = static_cast<int64_t>(nb_max) * ((max_suffix_len + BT_BN - 1) / BT_BN);
  int c = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(sm_count / units, BT_MAX_CTAS)));
  // no more CTAs than pairs of tiles a unit certainly has
  const int64_t t_min = Tp + (max_suffix_len + BT_BN - 1) / BT_BN;
  c = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(c, t_min / 2)));
  // the tile list of a CTA must fit its table
  if ((Tp + c - 1) / c + (Ts_max + c - 1) / c + 2 > BT_MAX_TILES) return pl;
  pl.row_tiles = static_cast<int>(row_tiles);
  pl.units = static_cast<int>(units);
  pl.ctas_per_unit = c;
  pl.ok = true;
  return pl;
}

static size_t bt_scratch_bytes(const BtPlan& pl) {
  if (pl.ctas_per_unit <= 1) return 0;
  return SCRATCH_COUNTER_BYTES +
         static_cast<size_t>(pl.units) * pl.ctas_per_unit * (BT_PART_FLOATS + BT_ML_FLOATS) * sizeof(float);
}

bool branch_tc_supported(const CacheView& suffix, int prefix_len, int max_suffix_len, int n_branches, int q_heads,
                         int q_len, float scale, int sm_count) {
  if (suffix.head_dim != BT_D || !(scale > 0.f) || !(scale < INFINITY) || encode_fn() == nullptr) return false;
  return bt_plan(prefix_len, max_suffix_len, n_branches, q_heads, suffix.kv_heads, q_len, sm_count).ok;
}

size_t branch_tc_workspace_bytes(int prefix_len, int max_suffix_len, int n_branches, int q_heads, int kv_heads,
                                 int q_len, int sm_count) {
  return bt_scratch_bytes(bt_plan(prefix_len, max_suffix_len, n_branches, q_heads, kv_heads, q_len, sm_count));
}

cudaError_t launch_branch_tc(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                             const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len,
                             int n_branches, int q_heads, int q_len, float scale, float* out, float* lse, int* status,
                             long long wait_limit, void* workspace, size_t workspace_bytes, cudaStream_t st,
                             LaunchInfo& li, const bf16* k_new, const bf16* v_new) {
  BtPlan pl = bt_plan(prefix_len, max_suffix_len, n_branches, q_heads, suffix.kv_heads, q_len, li.sm_count);
  if (!pl.ok) return cudaErrorInvalidValue;
  // several CTAs per unit need the scratch; with too little of it the units are not split
  while (pl.ctas_per_unit > 1 && (!workspace || bt_scratch_bytes(pl) > workspace_bytes)) pl.ctas_per_unit -= 1;
  const int G = q_heads / suffix.kv_heads;
  const uint64_t tokens = static_cast<uint64_t>(n_branches) * q_len;
  CUtensorMap tq, tpk, tpv, tsk, tsv, to;
  {  // q: [tokens][q_heads][128]; a box is [128 / G tokens][G heads][64 columns]: 128 stacked rows in order
    const uint64_t d[4] = {BT_D, static_cast<uint64_t>(q_heads), tokens, 1};
    const uint64_t s[3] = {BT_D * 2ull, static_cast<uint64_t>(q_heads) * BT_D * 2ull, 0};
    const uint32_t bx[4] = {64, static_cast<uint32_t>(G), static_cast<uint32_t>(BT_BM / G), 1};
    if (!make_map_bf16(&tq, q, d, s, bx)) return cudaErrorInvalidValue;
  }
  {  // out: same rows, fp32, boxes of 32 columns
    const uint64_t d[4] = {BT_D, static_cast<uint64_t>(q_heads), tokens, 1};
    const uint64_t s[3] = {BT_D * 4ull, static_cast<uint64_t>(q_heads) * BT_D * 4ull, 0};
    const uint32_t bx[4] = {32, static_cast<uint32_t>(G), static_cast<uint32_t>(BT_BM / G), 1};
    if (!make_map_f32(&to, out, d, s, bx)) return cudaErrorInvalidValue;
  }
  {  // suffix caches: rows at or beyond max_suffix_len read as zero
    const uint64_t d[4] = {BT_D, static_cast<uint64_t>(max_suffix_len), static_cast<uint64_t>(suffix.kv_heads),
                           static_cast<uint64_t>(suffix.batch)};
    const uint64_t s[3] = {static_cast<uint64_t>(suffix.sr) * 2, static_cast<uint64_t>(suffix.sh) * 2,
                           static_cast<uint64_t>(suffix.sb) * 2};
    const uint32_t bx[4] = {64, BT_BN, 1, 1};
    if (!make_map_bf16(&tsk, suffix.k, d, s, bx) || !make_map_bf16(&tsv, suffix.v, d, s, bx)) return cudaErrorInvalidValue;
  }
  if (prefix_len > 0) {  // rows at or beyond prefix_len read as zero
    const uint64_t d[4] = {BT_D, static_cast<uint64_t>(prefix_len), static_cast<uint64_t>(prefix.kv_heads), 1};
    const uint64_t s[3] = {static_cast<uint64_t>(prefix.sr) * 2, static_cast<uint64_t>(prefix.sh) * 2, 0};
    const uint32_t bx[4] = {64, BT_BN, 1, 1};
    if (!make_map_bf16(&tpk, prefix.k, d, s, bx) || !make_map_bf16(&tpv, prefix.v, d, s, bx)) return cudaErrorInvalidValue;
  } else {
    tpk = tsk;  // never dereferenced without a prefix
    tpv = tsv;
  }
  BtParams p;
  p.n_branches = n_branches;
  p.q_len = q_len;
  p.q_heads = q_heads;
  p.group = G;
  p.kv_heads = suffix.kv_heads;
  p.prefix_len = prefix_len;
  p.max_suffix_len = max_suffix_len;
  p.row_tiles = pl.row_tiles;
  p.ctas_per_unit = pl.ctas_per_unit;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.wait_limit = wait_limit;
  p.d_suffix_len = d_suffix_len;
  p.tree_mask = d_tree_mask;
  p.k_new = k_new;
  p.v_new = v_new;
  p.k_cache = const_cast<bf16*>(suffix.k);
  p.v_cache = const_cast<bf16*>(suffix.v);
  p.sb = suffix.sb;
  p.sh = suffix.sh;
  p.sr = suffix.sr;
  p.lse = lse;
  p.status = status;
  p.counters = static_cast<int*>(workspace);
  p.part = pl.ctas_per_unit > 1 ? reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + SCRATCH_COUNTER_BYTES)
                                : nullptr;
  p.ml = pl.ctas_per_unit > 1 ? p.part + static_cast<size_t>(pl.units) * pl.ctas_per_unit * BT_PART_FLOATS : nullptr;
  static PerDeviceOnce attr_done;
  if (!attr_done.done()) {
    cudaError_t e = cudaFuncSetAttribute(branch_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BT_SMEM_BYTES);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(branch_tc_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_done.set();
  }
  li.launches += 1;
  return launch_pdl(branch_tc_kernel, dim3(static_cast<unsigned>(pl.units * pl.ctas_per_unit)), dim3(BT_THREADS),
                    BT_SMEM_BYTES, st, tq, tpk, tpv, tsk, tsv, to, p);
}

}  // namespace jup
