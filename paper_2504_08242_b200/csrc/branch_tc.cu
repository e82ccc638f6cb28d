// Branch attention with many stacked query rows per kv head on the 5th-generation tensor cores (paper Sec. V-A,
// Fig. 7 step 3: the k draft tokens of every request are verified in one pass; Sec. V-B, Fig. 8: all
// point-extending requests share the prompt's KVCache).
//
// head_dim 128.  The stacked rows of a kv head -- (branch, draft token, head of the group), in that order -- are
// cut into row tiles of at most 128 rows: whole branches while a branch has at most 128 rows (the same number
// of branches in every tile, so that the tiles carry equal work), else 128-row slices of one branch.
// A unit = (kv head, row tile).  Every row belongs to one branch and may see the shared prefix plus that
// branch's suffix, so a row keeps ONE online-softmax state in its TMEM lane while the unit walks
//     prefix | suffix of the tile's first branch | ... | suffix of its last branch
// in tiles of 128 keys: a prefix tile is visible to every row, a suffix tile to the rows of its branch below
// their causal limit (or tree mask).  A prefix K/V tile is therefore fetched once per row tile, not once per branch.
//
// `ctas_per_unit` CTAs, a thread-block cluster, share a unit: the prefix tiles are cut into equal contiguous
// ranges, one per CTA, and so are the suffix tiles (the prefix share does not depend on the device-side lengths,
// so its first loads are in flight while the lengths arrive).  Inside a CTA:
//   loader warp  : TMA (tiled, 128-byte swizzle) Q once -- one box [tokens][G heads][64] lands in stacked-row
//                  order -- then the K/V tiles of the CTA's list into 3-stage rings, K and V refilled independently
//   patch warp   : passes landed tiles on to the MMA issuers, after patching those that need it: the last tiles of a
//                  branch's suffix hold rows that TMA cannot know about: rows at or beyond the device-side length
//                  (dead; their V rows are zeroed so that 0 x NaN never reaches an accumulator) and, with the fused
//                  KVCache write, the rows of this step's block, which are read from k_new / v_new into the tile
//                  (and stored into the cache by the unit that owns them)
//   MMA warps    : one thread per stream issues its tcgen05.mma  S = Q K^T  and  O += P V, accumulators in TMEM
//   softmax WGs  : two warpgroups run two independent online-softmax streams over the even and the odd tiles of
//                  the CTA's list (one thread per row); a warp none of whose rows sees a tile only zeroes its P
// TMEM (512 columns): S_0 | S_1 | O_0 | O_1.
// At the end the two streams of a CTA are merged in registers.  With one CTA per unit the rows are normalised
// and written out.  Otherwise every CTA writes its rows' unnormalised (O, m, l) to scratch (L2), and behind ONE
// cluster barrier CTA r of the cluster finishes a contiguous slice of the rows: it adds the partials in CTA
// order -- the result never depends on timing -- normalises and writes the output.  (Pushing the partials into the
// owner's shared memory instead was measured: 64 KB per CTA took 2.3 us over distributed shared memory, twice the
// trip through L2.)  No atomics, no second launch, nothing waits on a flag.
// All mbarrier waits are bounded; on expiry the CTA sets the status word, drains its own copies and MMAs,
// frees TMEM and returns (every thread still passes the cluster barriers).
#include <algorithm>
#include <atomic>

#include "host_checks.h"
#include "kernels.h"
#include "tc_common.cuh"
#include "tc_softmax.cuh"
#include "tmap.h"

namespace jup {

constexpr int BT_D = 128;
constexpr int BT_BM = 128;             // stacked rows per tile (at most)
constexpr int BT_BN = 128;             // keys per KV tile
constexpr int BT_TILE_BYTES = 32768;   // 128 x 128 bf16
constexpr int BT_PANEL_BYTES = 16384;  // 128 rows x 64 elements
constexpr int BT_KV_STAGES = 3;
constexpr int BT_MAX_BRANCHES = 32;    // branches in one row tile
constexpr int BT_MAX_CTAS = 8;         // CTAs per unit (the portable cluster size)
constexpr int BT_RECV_STRIDE = BT_D + 4;  // one CTA per unit: floats per staged row: O, then (m, l), padded against bank conflicts
constexpr int BT_PART_FLOATS = BT_BM * BT_D;  // one CTA's partial accumulator
constexpr int BT_ML_FLOATS = BT_BM * 2;       // and its (m, l) pairs

struct BtParams {
  int n_branches, q_len, q_heads, group, kv_heads;
  int prefix_len, max_suffix_len;
  int row_tiles;          // row tiles per kv head
  int branches_per_tile;  // whole branches per row tile (slices_per_branch == 1)
  int slices_per_branch;  // > 1: a branch has more than 128 rows and is cut into 128-row slices
  int box_tokens;         // tokens in the Q box
  int ctas_per_unit;      // cluster size
  float scale_log2;
  long long wait_limit;
  const int32_t* d_suffix_len;
  const uint32_t* tree_mask;  // nullable: [n_branches][q_len] ancestor bit masks of the draft block
  const bf16* k_new;          // nullable: fused KVCache write, [n_branches][q_len][kv_heads][128]
  const bf16* v_new;
  bf16* k_cache;              // the suffix cache (written only with the fused write)
  bf16* v_cache;
  int64_t sb, sh, sr;
  float* out;
  float* lse;
  int* status;
  float* part;  // ctas_per_unit > 1: [units][ctas_per_unit][32 column chunks][128 rows] float4, a CTA's partial accumulator
  float* ml;    //                    [units][ctas_per_unit][128 rows] (m, l)
};

// shared memory: [Q][K ring][V ring][barriers, flags][lengths and tile counts of the row tile's branches]
constexpr int BT_SMEM_Q = 0;
constexpr int BT_SMEM_K = BT_TILE_BYTES;
constexpr int BT_SMEM_V = BT_SMEM_K + BT_KV_STAGES * BT_TILE_BYTES;
constexpr int BT_SMEM_BAR = BT_SMEM_V + BT_KV_STAGES * BT_TILE_BYTES;
constexpr int BT_SMEM_LEN = BT_SMEM_BAR + 256;
constexpr int BT_SMEM_BYTES = BT_SMEM_LEN + 2 * BT_MAX_BRANCHES * 4 + 1024;  // + slack for 1024-byte alignment
static_assert(BT_SMEM_BYTES <= 227 * 1024, "shared memory per CTA");
static_assert(BT_BM * BT_RECV_STRIDE * 4 <= 2 * BT_KV_STAGES * BT_TILE_BYTES, "the staged rows fit in the rings");
constexpr int BT_LOADER_WARP = 8,  // warps 0..7: the two softmax warpgroups
              BT_MMA_WARP = 9,  // and 10: one issuer per stream
              BT_PATCH_WARP = 11;
constexpr int BT_THREADS = 32 * 12;

enum {
  BT_Q_FULL = 0,
  BT_K_FULL = 1,    // [3]
  BT_K_EMPTY = 4,   // [3]
  BT_V_FULL = 7,    // [3]
  BT_V_EMPTY = 10,  // [3]
  BT_S_FULL = 13,   // [2]
  BT_P_FULL = 15,   // [2]
  BT_O_READY = 17,  // [2]
  BT_DRAIN = 19,    // [2]
  BT_BAR_COUNT = 21
};

// One entry of a CTA's tile list.
struct BtTile {
  int seg;     // branch as an index into the row tile's branches; -1: the shared prefix
  int tile;    // tile number inside the segment
  bool patch;  // the patch warp has work on it
};

__global__ void __launch_bounds__(BT_THREADS, 1)
branch_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_pk,
                 const __grid_constant__ CUtensorMap tm_pv, const __grid_constant__ CUtensorMap tm_sk,
                 const __grid_constant__ CUtensorMap tm_sv, BtParams p) {
  constexpr int KV_STAGES = BT_KV_STAGES;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base + BT_SMEM_Q, sK = smem_base + BT_SMEM_K, sV = smem_base + BT_SMEM_V;
  const uint32_t sBar = smem_base + BT_SMEM_BAR;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + BT_SMEM_BAR + 8 * BT_BAR_COUNT);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + BT_SMEM_BAR + 8 * BT_BAR_COUNT + 8);
  volatile int* suffix_share = reinterpret_cast<volatile int*>(smem_gen + BT_SMEM_BAR + 8 * BT_BAR_COUNT + 16);  // [2]
  // how many K / V tiles of the list are ready for the tensor cores (landed and patched), published by the loader warp
  const uint32_t k_ready = sBar + 8 * BT_BAR_COUNT + 24, v_ready = k_ready + 4;
  int* len_s = reinterpret_cast<int*>(smem_gen + BT_SMEM_LEN);  // clamped suffix length of the tile's branches
  int* cum_s = len_s + BT_MAX_BRANCHES;                         // one past the last suffix tile of each
  auto bar = [&](int i) { return sBar + 8u * i; };
  const long long wl = p.wait_limit;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int C = p.ctas_per_unit;
  const int unit = blockIdx.x / C, crank = blockIdx.x % C;  // clusters are consecutive CTAs: crank is the cluster rank
  const int rt = unit % p.row_tiles, hk = unit / p.row_tiles;
  const int n = p.q_len, G = p.group;
  // ---- the row tile: tokens [tok0, tok0 + ntok) of the stacked (branch, draft row) order, all heads of the group
  int b_first, nb, tok0, ntok;
  if (p.slices_per_branch == 1) {
    b_first = rt * p.branches_per_tile;
    nb = min(p.branches_per_tile, p.n_branches - b_first);
    tok0 = b_first * n;
    ntok = nb * n;
  } else {
    b_first = rt / p.slices_per_branch;
    nb = 1;
    const int first = (rt % p.slices_per_branch) * (BT_BM / G);
    tok0 = b_first * n + first;
    ntok = min(BT_BM / G, n - first);
  }
  const int rows_here = ntok * G;
  const int P = p.prefix_len;
  const bool fused = p.k_new != nullptr;
  // this CTA's share of the prefix tiles: known without any memory access
  const int Tp = (P + BT_BN - 1) / BT_BN;
  const int p0 = Tp * crank / C, npre = Tp * (crank + 1) / C - p0;

  // ---- set-up
  if (threadIdx.x == 0) {
    for (int i = 0; i < BT_BAR_COUNT; ++i) mbar_init(bar(i), (i == BT_P_FULL || i == BT_P_FULL + 1) ? 128u : 1u);
    *abort_flag = 0;
    count_publish(k_ready, 0);
    count_publish(v_ready, 0);
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
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();  // everything above overlapped the previous kernel's tail; global memory is touched from here on

  auto load_k = [&](int s, const BtTile& e) {  // K of list entry e into the ring slot of sequence number s
    const int slot = s % KV_STAGES;
    const bool pre = e.seg < 0;
    const int row = e.tile * BT_BN, bb = pre ? 0 : b_first + e.seg;
    mbar_expect_tx(bar(BT_K_FULL + slot), BT_TILE_BYTES);
    const CUtensorMap* mk = pre ? &tm_pk : &tm_sk;
    tma_load_4d(sK + slot * BT_TILE_BYTES, mk, bar(BT_K_FULL + slot), 0, row, hk, bb);
    tma_load_4d(sK + slot * BT_TILE_BYTES + BT_PANEL_BYTES, mk, bar(BT_K_FULL + slot), 64, row, hk, bb);
  };
  auto load_v = [&](int s, const BtTile& e) {
    const int slot = s % KV_STAGES;
    const bool pre = e.seg < 0;
    const int row = e.tile * BT_BN, bb = pre ? 0 : b_first + e.seg;
    mbar_expect_tx(bar(BT_V_FULL + slot), BT_TILE_BYTES);
    const CUtensorMap* mv = pre ? &tm_pv : &tm_sv;
    tma_load_4d(sV + slot * BT_TILE_BYTES, mv, bar(BT_V_FULL + slot), 0, row, hk, bb);
    tma_load_4d(sV + slot * BT_TILE_BYTES + BT_PANEL_BYTES, mv, bar(BT_V_FULL + slot), 64, row, hk, bb);
  };
  const int pre_issued = min(npre, KV_STAGES);
  if (warp == BT_LOADER_WARP && lane == 0) {
    // Q: box_tokens tokens from tok0 on, heads hk G .. hk G + G - 1, one box per 64-column panel; the box lands as
    // rows (token, head) = stacked-row order.  Rows of the Q buffer beyond the box are never written: they belong
    // to no row of this tile and whatever the tensor cores make of them is never used.
    mbar_expect_tx(bar(BT_Q_FULL), static_cast<uint32_t>(p.box_tokens) * G * 256u);
    tma_load_4d(sQ, &tm_q, bar(BT_Q_FULL), 0, hk * G, tok0, 0);
    tma_load_4d(sQ + BT_PANEL_BYTES, &tm_q, bar(BT_Q_FULL), 64, hk * G, tok0, 0);
    for (int s = 0; s < pre_issued; ++s) {
      load_k(s, BtTile{-1, p0 + s, false});
      load_v(s, BtTile{-1, p0 + s, false});
    }
  } else if (warp == 0) {
    // ---- lengths and tile counts of the row tile's branches
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
    if (lane == 31) {  // this CTA's share of the unit's suffix tiles
      const int s0 = static_cast<int>(static_cast<int64_t>(cum) * crank / C);
      suffix_share[0] = s0;
      suffix_share[1] = static_cast<int>(static_cast<int64_t>(cum) * (crank + 1) / C) - s0;
    }
  }
  __syncthreads();
  const int s0 = suffix_share[0];
  const int Tall = npre + suffix_share[1];
  // Entry `s` of this CTA's list: its prefix share first, then its share of the suffix tiles of the row tile's
  // branches.  A role walks the list in increasing order and keeps the branch it has reached in `cursor`.
  auto tile_at = [&](int s, int& cursor) {
    if (s < npre) return BtTile{-1, p0 + s, false};
    const int g = s0 + (s - npre);
    while (cursor < nb - 1 && cum_s[cursor] <= g) ++cursor;
    const int tile = g - (cursor > 0 ? cum_s[cursor - 1] : 0);
    const int first_special = fused ? len_s[cursor] - n : len_s[cursor];  // first row that is new or dead
    return BtTile{cursor, tile, (tile + 1) * BT_BN > first_special};
  };
  const int T[2] = {(Tall + 1) >> 1, Tall >> 1};  // stream x takes the sequence numbers 2 i + x

  // a softmax thread's state after its last tile, kept for the merge behind the role branches
  float fin_m = -INFINITY, fin_l = 0.f, fin_w_own = 0.f, fin_w_oth = 0.f;

  if (warp == BT_LOADER_WARP) {
    // =============================================================== loader
    if (lane == 0) {
      // K and V rings are refilled independently: a K slot is free once its Q K^T has run, a V slot only after
      // its P V, and neither queue may hold up the other
      bool ok = true;
      int kn = pre_issued, vn = pre_issued, k_cursor = 0, v_cursor = 0;
      PollGuard guard(wl);
      while (ok && (kn < Tall || vn < Tall)) {
        bool progress = false;
        if (kn < Tall && (kn < KV_STAGES || mbar_test_wait(bar(BT_K_EMPTY + kn % KV_STAGES), (kn / KV_STAGES - 1) & 1))) {
          load_k(kn, tile_at(kn, k_cursor));
          ++kn;
          progress = true;
        }
        if (vn < Tall && (vn < KV_STAGES || mbar_test_wait(bar(BT_V_EMPTY + vn % KV_STAGES), (vn / KV_STAGES - 1) & 1))) {
          load_v(vn, tile_at(vn, v_cursor));
          ++vn;
          progress = true;
        }
        if (progress) guard.progress();
        else ok = guard.idle(abort_flag, p.status);
      }
      if (*abort_flag) {
        // wait (bounded) until every copy this thread started has landed before shared memory is released
        int dummy = 0;
        volatile int* none = &dummy;
        for (int s = max(0, kn - KV_STAGES); s < kn; ++s)
          mbar_wait(bar(BT_K_FULL + s % KV_STAGES), (s / KV_STAGES) & 1, none, nullptr);
        for (int s = max(0, vn - KV_STAGES); s < vn; ++s)
          mbar_wait(bar(BT_V_FULL + s % KV_STAGES), (s / KV_STAGES) & 1, none, nullptr);
        mbar_wait(bar(BT_Q_FULL), 0, none, nullptr);
      }
    }
    __syncwarp();
  } else if (warp == BT_PATCH_WARP) {
    // =============================================================== patcher
    // One warp-uniform event loop: lane 0 watches the K and the V tiles land (each ring in list order); a landed
    // tile is patched by the whole warp where it needs it and then passed on to the MMA issuers by publishing
    // the ring's count of ready tiles.
    // Patching.  K: the rows of this step's block come from k_new (dead rows need nothing: their scores are
    // masked).  V: the block's rows from v_new, and zeros in the dead rows so that 0 x NaN never reaches the
    // accumulator.  The block's rows go into the cache once per (branch, kv head): by the unit whose row tile
    // starts the branch.
    const bool writer = fused && (p.slices_per_branch == 1 || rt % p.slices_per_branch == 0);
    auto pass_on = [&](bool is_v, int s, int& cursor) {
      const int slot = s % KV_STAGES, u = s / KV_STAGES;
      const BtTile e = tile_at(s, cursor);
      bool landed = true;  // (lane 0 has seen the tile land)
      if (e.patch && (is_v || fused)) {
        // the other lanes observe the completed phase themselves before they touch the tile
        landed = lane == 0 || mbar_wait(bar((is_v ? BT_V_FULL : BT_K_FULL) + slot), u & 1, abort_flag, p.status, wl);
        landed = __all_sync(0xffffffffu, landed);
      }
      if (landed && e.patch && (is_v || fused)) {
        const int b = b_first + e.seg, L = len_s[e.seg], key0 = e.tile * BT_BN;
        const int new_begin = fused ? L - n : L;
        const int r_begin = max(new_begin - key0, 0);     // first row that is new or dead
        const int r_new = min(L - key0, BT_BN);           // rows [r_begin, r_new) are the block's, the rest is dead
        const bf16* fresh = is_v ? p.v_new : p.k_new;
        bf16* cache = is_v ? p.v_cache : p.k_cache;
        const uint32_t tile_addr = (is_v ? sV : sK) + slot * BT_TILE_BYTES;
        // 16-byte piece c of row r in the 128-byte-swizzled two-panel tile
        auto piece = [&](int r, int c) { return tile_addr + (c >> 3) * BT_PANEL_BYTES + r * 128 + (((c & 7) ^ (r & 7)) << 4); };
        // the block's rows: at most 16 rows x 16 pieces = 8 per lane, all loads in flight at once
        uint4 w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int idx = lane + 32 * k, r = r_begin + (idx >> 4), c = idx & 15;
          if (r < r_new)
            w[k] = __ldg(reinterpret_cast<const uint4*>(
                fresh + ((static_cast<int64_t>(b) * n + (key0 + r - new_begin)) * p.kv_heads + hk) * BT_D + c * 8));
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int idx = lane + 32 * k, r = r_begin + (idx >> 4), c = idx & 15;
          if (r < r_new) {
            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};\n" ::"r"(piece(r, c)), "r"(w[k].x), "r"(w[k].y),
                         "r"(w[k].z), "r"(w[k].w)
                         : "memory");
            if (writer)
              *reinterpret_cast<uint4*>(cache + b * p.sb + hk * p.sh + static_cast<int64_t>(key0 + r) * p.sr + c * 8) = w[k];
          }
        }
        if (is_v)
          for (int idx = lane; idx < (BT_BN - max(r_new, 0)) * 16; idx += 32)
            asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};\n" ::"r"(piece(max(r_new, 0) + (idx >> 4), idx & 15)), "r"(0u)
                         : "memory");
        fence_proxy_async();  // the tensor cores read the slot through the async proxy
      }
      __syncwarp();
      if (lane == 0 && landed) count_publish(is_v ? v_ready : k_ready, s + 1);
      return landed;
    };
    bool ok = true;
    int kp = 0, vp = 0, kp_cursor = 0, vp_cursor = 0;  // next tiles to pass on
    PollGuard guard(wl);
    while (ok && (kp < Tall || vp < Tall)) {
      int ev = 0;  // 1: K tile kp has landed; 2: V tile vp has landed
      if (lane == 0) {
        if (kp < Tall && mbar_test_wait(bar(BT_K_FULL + kp % KV_STAGES), (kp / KV_STAGES) & 1)) ev |= 1;
        if (vp < Tall && mbar_test_wait(bar(BT_V_FULL + vp % KV_STAGES), (vp / KV_STAGES) & 1)) ev |= 2;
      }
      ev = __shfl_sync(0xffffffffu, ev, 0);
      if (ev & 1) ok = pass_on(false, kp++, kp_cursor) && ok;
      if (ev & 2) ok = pass_on(true, vp++, vp_cursor) && ok;
      if (ev) guard.progress();
      else ok = guard.idle(abort_flag, p.status);
      ok = __shfl_sync(0xffffffffu, ok, 0);
    }
  } else if (warp == BT_MMA_WARP || warp == BT_MMA_WARP + 1) {
    // =============================================================== MMA issuers, one thread per stream
    // Stream x's order is fixed -- S(s) -> [softmax] -> P V(s) -> S(s + 2), the stream has one S buffer -- so its
    // issuer simply blocks on what comes next; the two streams never wait for each other.
    if (lane == 0) {
      const int x = warp - BT_MMA_WARP;
      constexpr uint32_t idesc_qk = tc_idesc_bf16(BT_BM, BT_BN, false, false);
      constexpr uint32_t idesc_pv = tc_idesc_bf16(BT_BM, BT_D, false, true);
      const uint32_t s_col = tmem + x * 128, o_col = tmem + 256 + x * 128;
      // descriptor halves (tc_desc_lo): one integer addition per operand slice keeps the issue loop short
      const uint32_t q_lo = tc_desc_lo(sQ, 16);
      auto issue_qk = [&](int s) {  // S = Q K^T, K of sequence number s
        const uint32_t k_lo = tc_desc_lo(sK + (s % KV_STAGES) * BT_TILE_BYTES, 16);
#pragma unroll
        for (int ks = 0; ks < BT_D / 16; ++ks) {
          const uint32_t off = ((ks >> 2) * BT_PANEL_BYTES + (ks & 3) * 32) >> 4;
          tc_mma_ss_lo(s_col, q_lo + off, k_lo + off, idesc_qk, ks > 0);
        }
      };
      auto issue_pv = [&](int s, bool first) {  // O (+)= P V, V of sequence number s
        const uint32_t v_lo = tc_desc_lo(sV + (s % KV_STAGES) * BT_TILE_BYTES, BT_PANEL_BYTES);
#pragma unroll
        for (int ks = 0; ks < BT_BN / 16; ++ks)
          tc_mma_ts_lo(o_col, s_col + ks * 8, v_lo + ks * (2048 >> 4), idesc_pv, (!first || ks > 0));
      };
      bool ok = mbar_wait(bar(BT_Q_FULL), 0, abort_flag, p.status, wl);  // (also when the list is empty: the copy must land)
      auto need_k = [&](int s) {
        ok = ok && count_wait(k_ready, s + 1, abort_flag, p.status, wl);
        tc_fence_after();
      };
      auto need_v = [&](int s) {
        ok = ok && count_wait(v_ready, s + 1, abort_flag, p.status, wl);
        tc_fence_after();
      };
      const int Tx = T[x];
      if (Tx > 0 && ok) {
        need_k(x);
        if (ok) {
          issue_qk(x);
          tc_commit(bar(BT_S_FULL + x));
          tc_commit(bar(BT_K_EMPTY + x % KV_STAGES));
        }
      }
      for (int j = 0; j < Tx && ok; ++j) {
        const int s = 2 * j + x, sn = s + 2;
        need_v(s);
        ok = ok && mbar_wait(bar(BT_P_FULL + x), j & 1, abort_flag, p.status, wl);
        if (!ok) break;
        tc_fence_after();
        issue_pv(s, j == 0);
        tc_commit(bar(BT_O_READY + x));
        tc_commit(bar(BT_V_EMPTY + s % KV_STAGES));
        if (j + 1 < Tx) {
          need_k(sn);
          if (!ok) break;
          issue_qk(sn);
          tc_commit(bar(BT_S_FULL + x));
          tc_commit(bar(BT_K_EMPTY + sn % KV_STAGES));
        }
      }
      if (!ok) {  // make sure no MMA of this thread is still running before TMEM and smem go away
        int dummy = 0;
        tc_commit(bar(BT_DRAIN + x));
        mbar_wait(bar(BT_DRAIN + x), 0, &dummy, nullptr);
      }
    }
    __syncwarp();
  } else {
    // =============================================================== softmax warpgroups (streams)
    const int x = warp >> 2;
    const int row_in_tile = (warp & 3) * 32 + lane;
    const bool row_valid = row_in_tile < rows_here;
    const int tok = tok0 + row_in_tile / G;          // token (branch, draft row) of this row
    const int rb = tok / n, ri = tok % n;
    const int rj = row_valid ? rb - b_first : -1;    // the row's branch as an index into the tile's branches
    // draft rows of the block this row may see, as bits: its ancestors and itself (a chain: rows 0..i)
    const uint32_t tm = !row_valid ? 0u
                        : (p.tree_mask ? __ldg(p.tree_mask + static_cast<int64_t>(rb) * n + ri) : (2u << ri) - 1u) &
                              ((1u << n) - 1u);
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + lane_base + x * 128;
    const uint32_t tO = tmem + lane_base + 256 + x * 128;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    int cursor = 0;
    const int Tx = T[x];
    for (int j = 0; j < Tx && ok; ++j) {
      // ---- which columns of the tile this row sees (a row beyond the tile's rows sees nothing); worked out while
      // the tensor cores still compute the tile's scores
      const BtTile e = tile_at(2 * j + x, cursor);
      const int key0 = e.tile * BT_BN;
      ColumnBits allow;
      bool full = false;
      if (e.seg < 0 && row_valid) {  // shared prefix: up to its end
        const int cnt = P - key0;
        full = cnt >= BT_BN;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int k = cnt - 32 * w;
          allow.w[w] = k >= 32 ? 0xffffffffu : (k <= 0 ? 0u : (1u << k) - 1u);
        }
      } else if (e.seg >= 0 && e.seg == rj) {  // the row's own branch: rows before the block, then the block by the mask
        const int hist = len_s[rj] - n - key0;  // column of the block's first row
        full = hist >= BT_BN;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          const int k = hist - 32 * w;
          const uint32_t before = k >= 32 ? 0xffffffffu : (k <= 0 ? 0u : (1u << k) - 1u);
          const uint32_t block = k >= 32 ? 0u : (k >= 0 ? tm << k : (k > -32 ? tm >> (-k) : 0u));
          allow.w[w] = before | block;
        }
      } else {  // another branch's suffix
        allow.w[0] = allow.w[1] = allow.w[2] = allow.w[3] = 0u;
      }
      const bool warp_sees = __any_sync(0xffffffffu, (allow.w[0] | allow.w[1] | allow.w[2] | allow.w[3]) != 0u);
      const bool masked = !__all_sync(0xffffffffu, full);
      ok = mbar_wait(bar(BT_S_FULL + x), j & 1, abort_flag, p.status, wl);
      if (!ok) break;
      tc_fence_after();
      auto wait_o = [&] { return mbar_wait(bar(BT_O_READY + x), (j - 1) & 1, abort_flag, p.status, wl); };
      if (warp_sees) {
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

    // ---- the two streams' (m, l) of a row cross through shared memory: the K slot of the stream's last tile,
    // free once its accumulator is complete; a stream without tiles owns slot x, never filled or long free
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
    fin_m = fmaxf(m_own, m_oth);
    fin_w_own = l > 0.f ? fast_exp2(m_own - fin_m) : 0.f;
    fin_w_oth = oth.y > 0.f ? fast_exp2(m_oth - fin_m) : 0.f;
    fin_l = l * fin_w_own + oth.y * fin_w_oth;
    if (C > 1) {
      // ---- this CTA's partial of the row -> scratch, as [column chunk][row] float4 so that a warp writes 512
      // contiguous bytes: columns [64 x, 64 x + 64) of both streams combined, unnormalised, relative to the row's
      // maximum over this CTA's tiles
      float4* gpart = reinterpret_cast<float4*>(p.part + (static_cast<size_t>(unit) * C + crank) * BT_PART_FLOATS);
      float2* gml = reinterpret_cast<float2*>(p.ml + (static_cast<size_t>(unit) * C + crank) * BT_ML_FLOATS);
      const bool has_own = Tx > 0, has_oth = T[1 - x] > 0;  // a stream without tiles never wrote its accumulator
      if ((warp & 3) * 32 < rows_here) {  // warp-uniform (the TMEM loads are warp-collective): the warp has a row
        const uint32_t tOwn = tmem + lane_base + 256 + x * 128 + x * 64;
        const uint32_t tOth = tmem + lane_base + 256 + (1 - x) * 128 + x * 64;
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
              v[i] = has_own ? __uint_as_float(o[4 * cc + i]) * fin_w_own : 0.f;
              if (has_oth) v[i] = fmaf(__uint_as_float(o2[4 * cc + i]), fin_w_oth, v[i]);
            }
            if (row_valid) gpart[(x * 16 + q2 * 8 + cc) * BT_BM + row_in_tile] = make_float4(v[0], v[1], v[2], v[3]);
          }
        }
        if (row_valid && x == 0) gml[row_in_tile] = make_float2(fin_l > 0.f ? fin_m : -INFINITY, fin_l);
      }
      __threadfence();  // visible to the cluster before its barrier is passed
    }
  }

  // ================================================================= output
  // Every thread of every CTA comes through here, whatever happened above.
  auto slice_begin = [&](int d) { return (BT_BM * d + C - 1) / C; };  // first row finished by CTA d of the cluster
  if (C > 1) {
    // ---- several CTAs per unit: behind the cluster barrier every CTA's partial is in the scratch (L2).  This CTA
    // finishes the rows [128 crank / C, 128 (crank + 1) / C).  First the normalised weight of every (CTA, row)
    // into shared memory, then (row, 16-byte column chunk) pairs dealt to the 256 threads with the row running
    // fastest (a warp reads contiguous pieces of every partial; a pair's loads are issued together, two pairs at a
    // time); the sums run in CTA order, so the result never depends on timing.
    tc_fence_before();
    cluster_sync_all();
    if (warp < 8) {
      const bool clean = *abort_flag == 0 && *reinterpret_cast<volatile int*>(p.status) == 0;  // nobody gave up on a wait
      const float2* uml = reinterpret_cast<const float2*>(p.ml + static_cast<size_t>(unit) * C * BT_ML_FLOATS);
      const float4* upart = reinterpret_cast<const float4*>(p.part + static_cast<size_t>(unit) * C * BT_PART_FLOATS);
      float* wtab = reinterpret_cast<float*>(smem_gen + BT_SMEM_K);  // [CTA][row of my slice] (the rings are free)
      const int row0 = slice_begin(crank), nrows = min(slice_begin(crank + 1), rows_here) - row0;
      const int max_slice = (BT_BM + C - 1) / C;
      if (static_cast<int>(threadIdx.x) < nrows) {
        const int row = row0 + threadIdx.x;
        float2 ml[BT_MAX_CTAS];
#pragma unroll
        for (int cr = 0; cr < BT_MAX_CTAS; ++cr)
          ml[cr] = cr < C ? __ldcg(uml + cr * BT_BM + row) : make_float2(-INFINITY, 0.f);
        float M = -INFINITY;
#pragma unroll
        for (int cr = 0; cr < BT_MAX_CTAS; ++cr)
          if (ml[cr].y > 0.f) M = fmaxf(M, ml[cr].x);  // a CTA whose tiles were all hidden from the row has l = 0
        float w[BT_MAX_CTAS], lall = 0.f;
#pragma unroll
        for (int cr = 0; cr < BT_MAX_CTAS; ++cr) {
          w[cr] = ml[cr].y > 0.f ? fast_exp2(ml[cr].x - M) : 0.f;
          lall = fmaf(w[cr], ml[cr].y, lall);
        }
        const float inv = 1.f / lall;
#pragma unroll
        for (int cr = 0; cr < BT_MAX_CTAS; ++cr)
          if (cr < C) wtab[cr * max_slice + threadIdx.x] = w[cr] * inv;
        if (clean && p.lse) {
          const int tok = tok0 + row / G, hq = hk * G + row % G;
          p.lse[(static_cast<int64_t>(tok / n) * p.q_heads + hq) * n + tok % n] = (M + log2f(lall)) * 0.69314718055994530942f;
        }
      }
      asm volatile("bar.sync 3, 256;\n" ::: "memory");
      const int pairs = nrows * 32;
      for (int idx0 = threadIdx.x; idx0 < pairs; idx0 += 512) {
        float4 t[2][BT_MAX_CTAS];
        int ris[2], chunk[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int idx = min(idx0 + h * 256, pairs - 1);
          ris[h] = idx % nrows;
          chunk[h] = idx / nrows;
#pragma unroll
          for (int cr = 0; cr < BT_MAX_CTAS; ++cr)
            if (cr < C)
              t[h][cr] = __ldcg(upart + static_cast<size_t>(cr) * (BT_PART_FLOATS / 4) + chunk[h] * BT_BM + row0 + ris[h]);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int cr = 0; cr < BT_MAX_CTAS; ++cr) {
            if (cr >= C) continue;
            const float w = wtab[cr * max_slice + ris[h]];
            if (w == 0.f) continue;  // (also a CTA without tiles, whose partial holds nothing meaningful)
            acc.x = fmaf(w, t[h][cr].x, acc.x);
            acc.y = fmaf(w, t[h][cr].y, acc.y);
            acc.z = fmaf(w, t[h][cr].z, acc.z);
            acc.w = fmaf(w, t[h][cr].w, acc.w);
          }
          if (clean && idx0 + h * 256 < pairs) {
            const int row = row0 + ris[h];
            const int tok = tok0 + row / G, hq = hk * G + row % G;
            *reinterpret_cast<float4*>(p.out + (static_cast<int64_t>(tok) * p.q_heads + hq) * BT_D + chunk[h] * 4) = acc;
          }
        }
      }
    }
  } else {
    // ---- one CTA per unit: the rows are staged in shared memory (every MMA and copy of the CTA is complete behind
    // the barrier, so the K/V rings are free) and written out as whole 512-byte rows
    float* stage = reinterpret_cast<float*>(smem_gen + BT_SMEM_K);  // [row][BT_RECV_STRIDE]
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp < 8 && (warp & 3) * 32 < rows_here) {  // warp-uniform (the TMEM loads are warp-collective)
      const int x = warp >> 2, row_in_tile = (warp & 3) * 32 + lane;
      const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
      const uint32_t tOwn = tmem + lane_base + 256 + x * 128 + x * 64;
      const uint32_t tOth = tmem + lane_base + 256 + (1 - x) * 128 + x * 64;
      const bool has_own = T[x] > 0, has_oth = T[1 - x] > 0;  // a stream without tiles never wrote its accumulator
      const float inv = 1.f / fin_l;
      const float a_own = fin_w_own * inv, a_oth = fin_w_oth * inv;
      float* dst = stage + row_in_tile * BT_RECV_STRIDE + x * 64;
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
            v[i] = has_own ? __uint_as_float(o[4 * cc + i]) * a_own : 0.f;
            if (has_oth) v[i] = fmaf(__uint_as_float(o2[4 * cc + i]), a_oth, v[i]);
          }
          *reinterpret_cast<float4*>(dst + q2 * 32 + cc * 4) = make_float4(v[0], v[1], v[2], v[3]);
        }
      }
      if (x == 0) *reinterpret_cast<float2*>(stage + row_in_tile * BT_RECV_STRIDE + BT_D) = make_float2(fin_m, fin_l);
    }
    __syncthreads();
    if (warp < 8) {
      const bool clean = *abort_flag == 0 && *reinterpret_cast<volatile int*>(p.status) == 0;  // nobody gave up on a wait
      for (int idx = threadIdx.x; idx < rows_here * 32 && clean; idx += 256) {
        const int row = idx >> 5, chunk = idx & 31;
        const int tok = tok0 + row / G, hq = hk * G + row % G;
        *reinterpret_cast<float4*>(p.out + (static_cast<int64_t>(tok) * p.q_heads + hq) * BT_D + chunk * 4) =
            *reinterpret_cast<const float4*>(stage + row * BT_RECV_STRIDE + chunk * 4);
        if (chunk == 0 && p.lse) {
          const float2 ml = *reinterpret_cast<const float2*>(stage + row * BT_RECV_STRIDE + BT_D);
          p.lse[(static_cast<int64_t>(tok / n) * p.q_heads + hq) * n + tok % n] =
              (ml.x + log2f(ml.y)) * 0.69314718055994530942f;
        }
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
  int row_tiles, branches_per_tile, slices_per_branch, box_tokens, units, ctas_per_unit;
  bool ok;
};

static cudaError_t bt_set_attributes() {
  static PerDeviceOnce attr_done;
  if (attr_done.done()) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(branch_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BT_SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(branch_tc_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess) attr_done.set();
  return e;
}

// How many clusters of c CTAs of the kernel can be resident at once on the current device (0 if the query fails).
static int bt_resident_clusters(int c) {
  static std::atomic<int> cache[64][BT_MAX_CTAS + 1];  // per device and cluster size: 0 = not asked yet, else answer + 1
  int dev = -1;
  if (c < 1 || c > BT_MAX_CTAS || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  const int cached = cache[dev][c].load(std::memory_order_acquire);
  if (cached > 0) return cached - 1;
  int n = 0;
  if (bt_set_attributes() == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(c * 64));
    cfg.blockDim = dim3(BT_THREADS);
    cfg.dynamicSmemBytes = BT_SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(c);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int got = 0;
    if (cudaOccupancyMaxActiveClusters(&got, branch_tc_kernel, &cfg) == cudaSuccess) n = got;
    else (void)cudaGetLastError();
  } else {
    (void)cudaGetLastError();
  }
  cache[dev][c].store(n + 1, std::memory_order_release);
  return n;
}

// The largest cluster size <= want whose clusters, one per unit, are all resident at once (1 if none is).
static int bt_cluster_size(int64_t units, int64_t want) {
  for (int c = static_cast<int>(std::min<int64_t>(want, BT_MAX_CTAS)); c >= 2; --c)
    if (bt_resident_clusters(c) >= units) return c;
  return 1;
}

static BtPlan bt_plan(int prefix_len, int max_suffix_len, int n_branches, int q_heads, int kv_heads, int q_len,
                      int sm_count) {
  BtPlan pl = {0, 0, 1, 0, 0, 1, false};
  const int G = q_heads / kv_heads, nG = q_len * G;
  const int64_t Tp = (static_cast<int64_t>(prefix_len) + BT_BN - 1) / BT_BN;
  const int64_t ts_max = (max_suffix_len + BT_BN - 1) / BT_BN;
  // CTAs per unit for a given number of units: fill the SMs, but no more CTAs than pairs of tiles a unit certainly has
  auto ctas_for = [&](int64_t units) {
    const int64_t want = std::min<int64_t>(std::max<int64_t>(sm_count / units, 1), std::max<int64_t>((Tp + ts_max) / 2, 1));
    return bt_cluster_size(units, want);
  };
  if (nG <= BT_BM) {
    // whole branches per row tile, the same number in every tile.  More, smaller tiles walk the prefix more often
    // but may fill the machine better: take the tiling with the shortest estimated walk per CTA (a branch's suffix
    // counted at 0.6 of its longest possible walk).
    const int per_tile_max = std::min(BT_MAX_BRANCHES, BT_BM / nG);
    const int tiles_min = (n_branches + per_tile_max - 1) / per_tile_max;
    const int64_t ts_est = std::max<int64_t>(1, (ts_max * 6 + 9) / 10);
    int64_t best = -1;
    for (int tiles = tiles_min; tiles <= std::min(n_branches, 2 * tiles_min); ++tiles) {
      const int per_tile = (n_branches + tiles - 1) / tiles;
      if (per_tile > per_tile_max || static_cast<int64_t>(tiles - 1) * per_tile >= n_branches) continue;
      const int64_t units = static_cast<int64_t>(tiles) * kv_heads;
      if (units > (1 << 30)) continue;
      const int c = ctas_for(units);
      const int64_t waves = (units * c + sm_count - 1) / sm_count;
      const int64_t est = waves * ((Tp + per_tile * ts_est + c - 1) / c + 3);  // + fixed cost of a CTA, in tiles
      if (best < 0 || est < best) {
        best = est;
        pl.row_tiles = tiles;
        pl.branches_per_tile = per_tile;
        pl.box_tokens = per_tile * q_len;
        pl.units = static_cast<int>(units);
        pl.ctas_per_unit = c;
      }
    }
    if (best < 0) return pl;
    pl.slices_per_branch = 1;
  } else {
    // a branch has more than 128 rows: 128-row slices, which must start on a token
    if (BT_BM % G != 0) return pl;
    pl.slices_per_branch = (nG + BT_BM - 1) / BT_BM;
    const int64_t tiles = static_cast<int64_t>(n_branches) * pl.slices_per_branch;
    const int64_t units = tiles * kv_heads;
    if (units > (1 << 30)) return pl;
    pl.row_tiles = static_cast<int>(tiles);
    pl.branches_per_tile = 1;
    pl.box_tokens = BT_BM / G;
    pl.units = static_cast<int>(units);
    pl.ctas_per_unit = ctas_for(units);
  }
  pl.ok = true;
  return pl;
}

static size_t bt_scratch_bytes(const BtPlan& pl) {
  if (pl.ctas_per_unit <= 1) return 0;
  return SCRATCH_COUNTER_BYTES +
         static_cast<size_t>(pl.units) * pl.ctas_per_unit * (BT_PART_FLOATS + BT_ML_FLOATS) * sizeof(float);
}

size_t branch_tc_workspace_bytes(int prefix_len, int max_suffix_len, int n_branches, int q_heads, int kv_heads,
                                 int q_len, int sm_count) {
  return bt_scratch_bytes(bt_plan(prefix_len, max_suffix_len, n_branches, q_heads, kv_heads, q_len, sm_count));
}

bool branch_tc_supported(const CacheView& suffix, int prefix_len, int max_suffix_len, int n_branches, int q_heads,
                         int q_len, float scale, int sm_count) {
  if (suffix.head_dim != BT_D || !(scale > 0.f) || !(scale < INFINITY) || encode_fn() == nullptr) return false;
  return bt_plan(prefix_len, max_suffix_len, n_branches, q_heads, suffix.kv_heads, q_len, sm_count).ok;
}

cudaError_t launch_branch_tc(const bf16* q, const CacheView& prefix, int prefix_len, const CacheView& suffix,
                             const int32_t* d_suffix_len, const uint32_t* d_tree_mask, int max_suffix_len,
                             int n_branches, int q_heads, int q_len, float scale, float* out, float* lse, int* status,
                             long long wait_limit, void* workspace, size_t workspace_bytes, cudaStream_t st,
                             LaunchInfo& li, const bf16* k_new, const bf16* v_new) {
  BtPlan pl = bt_plan(prefix_len, max_suffix_len, n_branches, q_heads, suffix.kv_heads, q_len, li.sm_count);
  if (!pl.ok) return cudaErrorInvalidValue;
  // several CTAs per unit exchange partials through the scratch; without enough of it a unit is walked by one CTA
  if (pl.ctas_per_unit > 1 && (!workspace || bt_scratch_bytes(pl) > workspace_bytes)) pl.ctas_per_unit = 1;
  const int G = q_heads / suffix.kv_heads;
  const uint64_t tokens = static_cast<uint64_t>(n_branches) * q_len;
  CUtensorMap tq, tpk, tpv, tsk, tsv;
  {  // q: [tokens][q_heads][128]; a box is [box_tokens tokens][G heads][64 columns]: the tile's stacked rows in order
    const uint64_t d[4] = {BT_D, static_cast<uint64_t>(q_heads), tokens, 1};
    const uint64_t s[3] = {BT_D * 2ull, static_cast<uint64_t>(q_heads) * BT_D * 2ull, 0};
    const uint32_t bx[4] = {64, static_cast<uint32_t>(G), static_cast<uint32_t>(pl.box_tokens), 1};
    if (!make_map_bf16(&tq, q, d, s, bx)) return cudaErrorInvalidValue;
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
  p.branches_per_tile = pl.branches_per_tile;
  p.slices_per_branch = pl.slices_per_branch;
  p.box_tokens = pl.box_tokens;
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
  p.out = out;
  p.lse = lse;
  p.status = status;
  p.part = pl.ctas_per_unit > 1 ? reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + SCRATCH_COUNTER_BYTES)
                                : nullptr;
  p.ml = pl.ctas_per_unit > 1 ? p.part + static_cast<size_t>(pl.units) * pl.ctas_per_unit * BT_PART_FLOATS : nullptr;
  cudaError_t e = bt_set_attributes();
  if (e != cudaSuccess) return e;
  li.launches += 1;
  return launch_pdl_cluster(branch_tc_kernel, dim3(static_cast<unsigned>(pl.units) * pl.ctas_per_unit), dim3(BT_THREADS),
                            BT_SMEM_BYTES, st, static_cast<unsigned>(pl.ctas_per_unit), tq, tpk, tpv, tsk, tsv, p);
}

}  // namespace jup
