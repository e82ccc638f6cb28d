// Chunked-prefill attention on the 5th-generation tensor cores (paper Sec. IV-A, Fig. 5(b)):
// chunk rows at positions pos..pos+n-1 attend causally to cache rows 0..pos+i.  head_dim 128.
//
// Two kernels, chosen by the size of the grid (see launch_tc):
//  - prefill_tc_kernel (this file): one CTA owns TWO query tiles of 128 rows of one (sequence, query head) and walks
//    the KV cache in tiles of 128 keys, every K/V tile serving both query tiles:
//      loader warp : TMA (tiled, 128-byte swizzle) Q once, then K/V tiles into 2-stage rings
//      MMA warp    : one thread issues tcgen05.mma  S = Q K^T  and  O += P V, accumulators in TMEM
//      softmax WGs : one warpgroup per query tile, one thread per row holding the row's 128 scores in registers:
//                    row maximum, P = exp2(...) with fp32-pair arithmetic written back over S as bf16 and released
//                    to the MMA issuer in two parts; lazy rescale of O only when the maximum grew by > 2^8
//    TMEM (512 columns): S_A | S_B | O_A | O_B (128 each).  For grids that cannot fill the SMs a cluster of 4 CTAs
//    shares the pair of query tiles and splits the KV walk (template parameter CL).
//  - prefill_frag_kernel (prefill_tc_frag.cuh): one query tile per CTA, both warpgroups on it.
// All mbarrier waits are bounded; on expiry the CTA sets the status word, drains its own copies and MMAs, frees
// TMEM and returns.
#include "host_checks.h"
#include <atomic>

#include "kernels.h"
#include "tc_common.cuh"
#include "tc_softmax.cuh"
#include "tmap.h"

namespace jup {

constexpr int TC_D = 128;
constexpr int TC_BM = 128;              // query rows per tile
constexpr int TC_BN = 128;              // keys per KV tile
constexpr int TC_TILE_BYTES = 32768;    // 128 x 128 bf16
constexpr int TC_PANEL_BYTES = 16384;   // 128 rows x 64 elements
constexpr int TC_CLUSTER_MIN_TILES = 18;     // shortest KV walk (in tiles) that a cluster of 4 CTAs shares

struct TcParams {
  int q_heads, group, q_len, pos, batch;
  int prefix_len;  // rows of a shared prefix cache attended before the sequence's own cache (0: none)
  int q_blocks;  // query tiles (fragment form) or pairs of query tiles per (sequence, head)
  float scale_log2;
  float* out;
  float* lse;
  int* status;
  float* scratch;  // cluster mode: per cluster, CL x (partial accumulators 2 x 128 x 128, then (m, l) 2 x 128 x 2)
  int prefix_batched;  // 1: the front segment has one cache per sequence (fused form), 0: one cache shared by all
  // Fused KVCache write (fused_write != 0).  The chunk's K/V rows, token-major [batch][q_len][kv_heads][128], are
  // the attention's own segment; the CTAs of each group's first query head also write them, bit-exactly, into rows
  // copy_pos + r of the cache, with tiled stores straight from the K/V slots the tiles were loaded into (tensor
  // maps tm_ck / tm_cv over the destination cache).
  int fused_write;
  int copy_pos;
};
constexpr int TC_PART_FLOATS = 2 * TC_BM * TC_D;  // one CTA's partial accumulators (both query tiles)
constexpr int TC_ML_FLOATS = 2 * TC_BM * 2;       // one CTA's (m, l) pairs

constexpr int TC_NQ = 2;  // query tiles per CTA
struct TcCfg {
  static constexpr int KV_STAGES = 2;
  static constexpr int SOFTMAX_WARPS = 4 * TC_NQ;
  static constexpr int LOADER_WARP = SOFTMAX_WARPS;
  static constexpr int MMA_WARP = SOFTMAX_WARPS + 1;
  // Three full warpgroups (the third: loader, MMA issuer, two idle warps) so that the register file can be
  // re-divided: a softmax thread holds a whole score row (REGS_SOFTMAX), the third warpgroup gives its share back
  // (REGS_OTHER); 2 x 128 x 208 + 128 x 88 = 384 x 168, the registers the CTA starts with.
  static constexpr int THREADS = 384;
  static constexpr int REGS_SOFTMAX = 208, REGS_OTHER = 88;
  static constexpr int O_COL0 = 256;
  // shared memory: [Q tiles][K ring][V ring][barriers]
  static constexpr int SMEM_Q = 0;
  static constexpr int SMEM_K = TC_NQ * TC_TILE_BYTES;
  static constexpr int SMEM_V = SMEM_K + KV_STAGES * TC_TILE_BYTES;
  static constexpr int SMEM_BAR = SMEM_V + KV_STAGES * TC_TILE_BYTES;
  static constexpr int SMEM_BYTES = SMEM_BAR + 256 + 1024;  // + slack for 1024-byte alignment
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory per CTA");
};

// barrier indices (8 bytes each) inside the barrier block
enum {
  BAR_Q_FULL = 0,    // [2]
  BAR_K_FULL = 2,    // [2]
  BAR_K_EMPTY = 4,   // [2]
  BAR_V_FULL = 6,    // [2]
  BAR_V_EMPTY = 8,   // [2]
  BAR_S_FULL = 10,   // [2] one per query tile
  BAR_P_FULL = 12,   // [2]
  BAR_O_READY = 14,  // [2]
  BAR_P_EARLY = 16,  // [2] the first 96 columns of P are in TMEM
  BAR_DRAIN = 18,
  BAR_COUNT = 19
};

constexpr int TC_BOX_FLOATS = TC_BM * 32;  // 16 KB
constexpr int NQ = TC_NQ;

// CL > 1: a thread-block cluster of CL CTAs shares one pair of query tiles; CTA r takes the KV tiles
// r, r + CL, r + 2 CL, ... and the partial (O, m, l) are exchanged through global scratch (L2) around one
// cluster barrier: distributed shared memory moved them at about 20 GB/s per SM when measured, L2 is
// several times faster.  CTA r then finishes the output columns [128 r / CL, 128 (r + 1) / CL).
template <int CL>
__global__ void __launch_bounds__(TcCfg::THREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_pk,
                  const __grid_constant__ CUtensorMap tm_pv, const __grid_constant__ CUtensorMap tm_o,
                  const __grid_constant__ CUtensorMap tm_ck, const __grid_constant__ CUtensorMap tm_cv, TcParams p) {
  using Cfg = TcCfg;
  constexpr int KV_STAGES = Cfg::KV_STAGES;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base + Cfg::SMEM_Q, sK = smem_base + Cfg::SMEM_K, sV = smem_base + Cfg::SMEM_V;
  const uint32_t sBar = smem_base + Cfg::SMEM_BAR;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + Cfg::SMEM_BAR + 8 * BAR_COUNT);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + Cfg::SMEM_BAR + 8 * BAR_COUNT + 8);
  auto bar = [&](int i) { return sBar + 8u * i; };

  // a CTA of a cluster can meet rows that see none of a tile, and ends with unnormalised partials
  constexpr bool PARTIAL = CL > 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int crank = CL > 1 ? static_cast<int>(cluster_ctarank()) : 0;

  // ---- work assignment: heaviest query blocks first
  const int nbh = p.batch * p.q_heads;
  const int work = blockIdx.x / CL;
  const int bh = work % nbh;
  const int qblk = p.q_blocks - 1 - work / nbh;
  const int b = bh / p.q_heads, h = bh % p.q_heads, hk = h / p.group;
  // KV tiles 0..Tp-1 come from the shared prefix (every row sees them, no causal limit), the rest from
  // the sequence's own cache
  const int Tp = (p.prefix_len + TC_BN - 1) / TC_BN;
  // T[x]: KV tiles of query tile x; Tall: KV tiles the CTA loads (its load sequence 0..Tall-1).  CTA r of a
  // cluster loads KV tile r + CL n as its n-th.
  int T[2] = {0, 0};
  int Tg[2] = {0, 0};  // cluster mode: tiles of the query tile over the whole cluster
#pragma unroll
  for (int x = 0; x < NQ; ++x) {
    const int r0 = (qblk * NQ + x) * TC_BM;
    if (r0 < p.q_len) T[x] = Tp + (p.pos + min(p.q_len, r0 + TC_BM) + TC_BN - 1) / TC_BN;
  }
  if constexpr (CL > 1) {
#pragma unroll
    for (int x = 0; x < NQ; ++x) {
      Tg[x] = T[x];
      T[x] = T[x] > crank ? (T[x] - crank + CL - 1) / CL : 0;
    }
  }
  const int Tall = max(T[0], T[1]);
  auto tile_of_seq = [&](int n) { return CL > 1 ? crank + CL * n : n; };  // KV tile of a sequence number

  // ---- set-up
  if (threadIdx.x == 0) {
    for (int i = 0; i < BAR_COUNT; ++i) mbar_init(bar(i), (i == BAR_P_FULL || i == BAR_P_FULL + 1 || i == BAR_P_EARLY || i == BAR_P_EARLY + 1) ? 128u : 1u);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == Cfg::MMA_WARP) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish();
  } else if (warp == Cfg::LOADER_WARP && lane == 0) {
    // the tensor maps are kernel parameters: fetching them does not depend on the previous kernel
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
    if (CL == 1) tma_prefetch_desc(&tm_o);
    if (Tp > 0) {
      tma_prefetch_desc(&tm_pk);
      tma_prefetch_desc(&tm_pv);
    }
    if (p.fused_write != 0) {
      tma_prefetch_desc(&tm_ck);
      tma_prefetch_desc(&tm_cv);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();  // everything above overlapped the previous kernel's tail; global memory is touched from here on

  float part_m = -INFINITY, part_l = 0.f;  // cluster mode: a softmax thread's (m, l) after its last tile

  if (warp == Cfg::LOADER_WARP) {
    // =============================================================== loader
    reg_dec<Cfg::REGS_OTHER>();
    if (lane == 0) {
#pragma unroll
      for (int x = 0; x < NQ; ++x) {
        if (T[x] == 0) continue;
        const int r0 = (qblk * NQ + x) * TC_BM;
        mbar_expect_tx(bar(BAR_Q_FULL + x), TC_TILE_BYTES);
        tma_load_4d(sQ + x * TC_TILE_BYTES, &tm_q, bar(BAR_Q_FULL + x), 0, h, r0, b);
        tma_load_4d(sQ + x * TC_TILE_BYTES + TC_PANEL_BYTES, &tm_q, bar(BAR_Q_FULL + x), 64, h, r0, b);
      }
      int issued = 0;
      bool ok = true;
      // Fused KVCache write: the chunk's own K/V tiles are loaded for the attention anyway; the tiles that hold
      // the query rows of this CTA (of this cluster: the CTA that loads them) go from their slots to the cache with
      // tiled stores, as soon as they have landed.  A slot is refilled only after its store has read it.
      constexpr int QT = NQ;  // query tiles of the chunk per CTA (cluster)
      const bool writer = p.fused_write != 0 && h % p.group == 0;
      auto store_own_tile = [&](int j) {  // j: load sequence number
        const int t = tile_of_seq(j) - Tp;  // tile of the chunk
        if (!writer || t < 0 || t / QT != qblk || t * TC_BN >= p.q_len) return;
        const int s = j % KV_STAGES, u = j / KV_STAGES;
        ok = ok && mbar_wait(bar(BAR_K_FULL + s), u & 1, abort_flag, p.status);
        ok = ok && mbar_wait(bar(BAR_V_FULL + s), u & 1, abort_flag, p.status);
        if (!ok) return;
        const int row = p.copy_pos + t * TC_BN;  // rows beyond copy_pos + q_len are clipped by the tensor maps
        tma_store_4d(&tm_ck, sK + s * TC_TILE_BYTES, 0, row, hk, b);
        tma_store_4d(&tm_ck, sK + s * TC_TILE_BYTES + TC_PANEL_BYTES, 64, row, hk, b);
        tma_store_4d(&tm_cv, sV + s * TC_TILE_BYTES, 0, row, hk, b);
        tma_store_4d(&tm_cv, sV + s * TC_TILE_BYTES + TC_PANEL_BYTES, 64, row, hk, b);
        tma_store_commit();
        tma_store_wait_read();
      };
      for (int j = 0; j < Tall && ok; ++j) {
        const int s = j % KV_STAGES, u = j / KV_STAGES;
        if (u > 0) store_own_tile(j - KV_STAGES);
        if (!ok) break;
        if (u > 0) ok = mbar_wait(bar(BAR_K_EMPTY + s), (u - 1) & 1, abort_flag, p.status);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_K_FULL + s), TC_TILE_BYTES);
        const int g = tile_of_seq(j);
        const CUtensorMap* mk = g < Tp ? &tm_pk : &tm_k;
        const int krow = (g < Tp ? g : g - Tp) * TC_BN, kb = (g < Tp && !p.prefix_batched) ? 0 : b;
        tma_load_4d(sK + s * TC_TILE_BYTES, mk, bar(BAR_K_FULL + s), 0, krow, hk, kb);
        tma_load_4d(sK + s * TC_TILE_BYTES + TC_PANEL_BYTES, mk, bar(BAR_K_FULL + s), 64, krow, hk, kb);
        if (u > 0) ok = mbar_wait(bar(BAR_V_EMPTY + s), (u - 1) & 1, abort_flag, p.status);
        if (!ok) {
          issued = 2 * j + 1;
          break;
        }
        mbar_expect_tx(bar(BAR_V_FULL + s), TC_TILE_BYTES);
        const CUtensorMap* mv = g < Tp ? &tm_pv : &tm_v;
        tma_load_4d(sV + s * TC_TILE_BYTES, mv, bar(BAR_V_FULL + s), 0, krow, hk, kb);
        tma_load_4d(sV + s * TC_TILE_BYTES + TC_PANEL_BYTES, mv, bar(BAR_V_FULL + s), 64, krow, hk, kb);
        issued = 2 * j + 2;
      }
      for (int j = max(0, Tall - KV_STAGES); j < Tall && ok; ++j) store_own_tile(j);
      if (*abort_flag) {
        // wait (bounded) until every copy this thread started has landed before shared memory is released
        int dummy = 0;
        volatile int* none = &dummy;
        const int nk = (issued + 1) / 2, nv = issued / 2;
        for (int j = max(0, nk - KV_STAGES); j < nk; ++j)
          mbar_wait(bar(BAR_K_FULL + j % KV_STAGES), (j / KV_STAGES) & 1, none, nullptr);
        for (int j = max(0, nv - KV_STAGES); j < nv; ++j)
          mbar_wait(bar(BAR_V_FULL + j % KV_STAGES), (j / KV_STAGES) & 1, none, nullptr);
        for (int x = 0; x < NQ; ++x)
          if (T[x] > 0) mbar_wait(bar(BAR_Q_FULL + x), 0, none, nullptr);
      }
    }
    __syncwarp();
  } else if (warp == Cfg::MMA_WARP) {
    // =============================================================== MMA issuer
    reg_dec<Cfg::REGS_OTHER>();
    if (lane == 0) {
      constexpr uint32_t idesc_qk = tc_idesc_bf16(TC_BM, TC_BN, false, false);
      constexpr uint32_t idesc_pv = tc_idesc_bf16(TC_BM, TC_D, false, true);
      auto s_col = [&](int x) { return tmem + x * 128; };
      auto o_col = [&](int x) { return tmem + Cfg::O_COL0 + x * 128; };
      // The issue loops are kept to an integer addition or two per MMA (descriptor halves, see tc_desc_lo): this
      // thread shares its scheduler with two softmax warps, and a longer chain of address arithmetic per MMA
      // made the issue, not the tensor pipe, the limit.
      auto issue_qk = [&](int x, int g) {  // S(x) = Q(x) K^T, K of load sequence number g
        const uint32_t q_lo = tc_desc_lo(sQ + x * TC_TILE_BYTES, 16);
        const uint32_t k_lo = tc_desc_lo(sK + (g % KV_STAGES) * TC_TILE_BYTES, 16);
        const uint32_t d = s_col(x);
#pragma unroll
        for (int ks = 0; ks < TC_D / 16; ++ks) {
          const uint32_t off = ((ks >> 2) * TC_PANEL_BYTES + (ks & 3) * 32) >> 4;
          tc_mma_ss_lo(d, q_lo + off, k_lo + off, idesc_qk, ks > 0);
        }
      };
      // O(x) (+)= P(x) V over the keys [16 ks0, 16 ks1) of the tile, V of load sequence number g
      auto issue_pv = [&](int x, int g, bool first, int ks0, int ks1) {
        const uint32_t v_lo = tc_desc_lo(sV + (g % KV_STAGES) * TC_TILE_BYTES, TC_PANEL_BYTES);
        const uint32_t d = o_col(x), a = s_col(x);
#pragma unroll
        for (int ks = ks0; ks < ks1; ++ks)
          tc_mma_ts_lo(d, a + ks * 8, v_lo + ks * (2048 >> 4), idesc_pv, (!first || ks > 0));
      };
      auto last_user = [&](int g) {  // the last query tile (in issue order) that uses the tile of sequence number g
        int r = -1;
#pragma unroll
        for (int x = 0; x < NQ; ++x)
          if (g < T[x]) r = x;
        return r;
      };
      bool ok = true;
      int k_waited = -1, v_waited = -1;
      auto need_k = [&](int j) {
        if (k_waited < j) {
          ok = ok && mbar_wait(bar(BAR_K_FULL + j % KV_STAGES), (j / KV_STAGES) & 1, abort_flag, p.status);
          k_waited = j;
          tc_fence_after();
        }
      };
      auto need_v = [&](int j) {
        if (v_waited < j) {
          ok = ok && mbar_wait(bar(BAR_V_FULL + j % KV_STAGES), (j / KV_STAGES) & 1, abort_flag, p.status);
          v_waited = j;
          tc_fence_after();
        }
      };
      // prologue: S(x, 0)
#pragma unroll
      for (int x = 0; x < NQ; ++x) {
        if (T[x] == 0 || !ok) continue;
        ok = ok && mbar_wait(bar(BAR_Q_FULL + x), 0, abort_flag, p.status);
        need_k(0);
        if (!ok) break;
        issue_qk(x, 0);
        tc_commit(bar(BAR_S_FULL + x));
        if (x == last_user(0)) tc_commit(bar(BAR_K_EMPTY + 0));
      }
      for (int j = 0; j < Tall && ok; ++j) {
#pragma unroll
        for (int x = 0; x < NQ; ++x) {
          if (j >= T[x] || !ok) continue;
          const int g = j, gn = j + 1;  // load sequence numbers
          need_v(g);
          ok = ok && mbar_wait(bar(BAR_P_EARLY + x), j & 1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_pv(x, g, j == 0, 0, 6);  // the first 96 keys while the softmax finishes the last 32
          ok = ok && mbar_wait(bar(BAR_P_FULL + x), j & 1, abort_flag, p.status);
          if (!ok) break;
          tc_fence_after();
          issue_pv(x, g, j == 0, 6, 8);
          tc_commit(bar(BAR_O_READY + x));
          if (x == last_user(g)) tc_commit(bar(BAR_V_EMPTY + g % KV_STAGES));
          if (j + 1 < T[x]) {
            need_k(gn);
            if (!ok) break;
            issue_qk(x, gn);
            tc_commit(bar(BAR_S_FULL + x));
            if (x == last_user(gn)) tc_commit(bar(BAR_K_EMPTY + gn % KV_STAGES));
          }
        }
      }
      if (!ok) {  // make sure no MMA of this thread is still running before TMEM and smem go away
        int dummy = 0;
        tc_commit(bar(BAR_DRAIN));
        mbar_wait(bar(BAR_DRAIN), 0, &dummy, nullptr);
      }
    }
    __syncwarp();
  } else if (warp < Cfg::SOFTMAX_WARPS) {
    // =============================================================== softmax warpgroups
    reg_inc<Cfg::REGS_SOFTMAX>();
    const int x = warp >> 2;                      // query tile of this warpgroup
    const int row_in_tile = (warp & 3) * 32 + lane;
    const int row = (qblk * NQ + x) * TC_BM + row_in_tile;  // row inside the chunk
    const bool row_valid = row < p.q_len;
    const int lim = p.pos + min(row, p.q_len - 1) + 1;      // keys j < lim are visible
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tO = tmem + lane_base + Cfg::O_COL0 + x * 128;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    const int Tx = T[x];
    for (int j = 0; j < Tx && ok; ++j) {
      const uint32_t tS = tmem + lane_base + x * 128;
      ok = mbar_wait(bar(BAR_S_FULL + x), j & 1, abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      // columns >= nvalid are masked: the end of the prefix in its last tile, the causal limit afterwards
      const int g = tile_of_seq(j);
      const int nvalid = g < Tp ? p.prefix_len - g * TC_BN : lim - (g - Tp) * TC_BN;
      // warp-uniform flag, so the warp stays converged for the collective tcgen05 operations
      const bool masked = __any_sync(0xffffffffu, nvalid < TC_BN);
      // (the accumulator's barrier is only consulted when O has to be rescaled: phase j - 1 cannot be overtaken,
      // because PV(j) needs this thread's P(j))
      ok = softmax_tile_row<PARTIAL>(
          tS, tO, j, masked, ColumnLimit{nvalid}, c, m_ref, l,
          [&] { return mbar_wait(bar(BAR_O_READY + x), (j - 1) & 1, abort_flag, p.status); },
          [&] {
            tc_fence_before();
            mbar_arrive(bar(BAR_P_EARLY + x));
          });
      if (!ok) break;
      tc_fence_before();
      mbar_arrive(bar(BAR_P_FULL + x));
    }
    pdl_launch_dependents();  // the next kernel of the stream may start its own set-up now
    if constexpr (CL > 1) {
      // the accumulator is complete; the merge over the cluster follows the role branches
      if (Tx > 0) ok = mbar_wait(bar(BAR_O_READY + x), (Tx - 1) & 1, abort_flag, p.status) && ok;
      part_m = m_ref;
      part_l = l;
    } else if (Tx > 0) {  // warpgroup-uniform: every thread of the tile reaches the named barriers below, even
                          // one that gave up on a wait (it only skips its global stores)
      ok = ok && mbar_wait(bar(BAR_O_READY + x), (Tx - 1) & 1, abort_flag, p.status);
      tc_fence_after();
      // O / l goes out through shared memory (this tile's Q buffer, free now) and tiled stores: two rounds of
      // two boxes of 128 rows x 32 columns; rows at or beyond q_len are clipped by the tensor map.
      const float inv = 1.f / l;
      float* stage = reinterpret_cast<float*>(smem_gen + Cfg::SMEM_Q + x * TC_TILE_BYTES);
      const uint32_t stage_addr = sQ + x * TC_TILE_BYTES;
      const int tid_t = threadIdx.x & 127;
      const int tile_row0 = (qblk * NQ + x) * TC_BM;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
        for (int q2 = 0; q2 < 2; ++q2) {
          uint32_t o[32];
          tmem_ld32(tO + hh * 64 + q2 * 32, o);
          tc_wait_ld();
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(o[i]) * inv;
          stage_box_row(stage + q2 * TC_BOX_FLOATS, row_in_tile, v);
        }
        fence_proxy_async();
        asm volatile("bar.sync %0, 128;\n" ::"r"(1 + x) : "memory");
        if (tid_t == 0) {
          if (ok) {
            tma_store_4d(&tm_o, stage_addr, hh * 64, h, tile_row0, b);
            tma_store_4d(&tm_o, stage_addr + TC_BOX_FLOATS * 4, hh * 64 + 32, h, tile_row0, b);
            tma_store_commit();
          }
          tma_store_wait_read();  // the boxes are rewritten next / shared memory is released at the end of the kernel
        }
        if (hh == 0) asm volatile("bar.sync %0, 128;\n" ::"r"(1 + x) : "memory");
      }
      if (ok && p.lse && row_valid)
        p.lse[(static_cast<int64_t>(b) * p.q_heads + h) * p.q_len + row] =
            (m_ref + log2f(l)) * 0.69314718055994530942f;
    }
  }

  else {
    reg_dec<Cfg::REGS_OTHER>();  // the idle warps of the third warpgroup: the re-division is a warpgroup's decision
  }

  if constexpr (CL > 1) {
    // ---- merge over the cluster.  Every thread of every CTA comes through here, whatever happened above.
    // Each softmax thread has seen its stream's last accumulator, so after this barrier every MMA of the
    // CTA is complete and every copy has landed: the K/V rings are free.
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    constexpr int W = TC_D / CL;  // output columns this CTA finishes
    // Partial accumulators, unnormalised fp32: [column slice CL][query tile 2][row 128][W], the 16-byte chunks
    // of a row XOR-swizzled by the row (bank conflicts); staged in the K/V rings, copied as they are to the
    // cluster's scratch.  (m, l) per row: [query tile 2][row 128].
    float* part = reinterpret_cast<float*>(smem_gen + Cfg::SMEM_K);
    static_assert(TC_PART_FLOATS * 4 <= 2 * KV_STAGES * TC_TILE_BYTES, "partials fit in the K/V rings");
    float* gpart = p.scratch + static_cast<size_t>(work) * CL * (TC_PART_FLOATS + TC_ML_FLOATS);
    float* gml = gpart + CL * TC_PART_FLOATS;
    if (warp < Cfg::SOFTMAX_WARPS) {
      const int x = warp >> 2, row_in_tile = (warp & 3) * 32 + lane;
      const uint32_t tO = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16) + Cfg::O_COL0 + x * 128;
      reinterpret_cast<float2*>(gml + crank * TC_ML_FLOATS)[x * TC_BM + row_in_tile] = make_float2(part_m, part_l);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t o[32];
        if (T[x] > 0) {  // warpgroup-uniform; a stream without tiles never wrote its accumulator
          tmem_ld32(tO + q4 * 32, o);
          tc_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = 0u;
        }
        const int slice = (q4 * 32) / W, chunk0 = ((q4 * 32) % W) / 4;
        float* dst = part + ((slice * 2 + x) * TC_BM + row_in_tile) * W;
#pragma unroll
        for (int cc = 0; cc < 8; ++cc)
          *reinterpret_cast<float4*>(dst + (((chunk0 + cc) ^ (row_in_tile & 7)) << 2)) =
              make_float4(__uint_as_float(o[4 * cc]), __uint_as_float(o[4 * cc + 1]), __uint_as_float(o[4 * cc + 2]),
                          __uint_as_float(o[4 * cc + 3]));
      }
      asm volatile("bar.sync 3, 256;\n" ::: "memory");
      const float4* src = reinterpret_cast<const float4*>(part);
      float4* dst = reinterpret_cast<float4*>(gpart + crank * TC_PART_FLOATS);
#pragma unroll 8
      for (int i = 0; i < TC_PART_FLOATS / 4 / 256; ++i) dst[i * 256 + threadIdx.x] = src[i * 256 + threadIdx.x];
      __threadfence();
    }
    cluster_sync_all();  // release / acquire over the cluster: the partials of every CTA are visible
    if (warp < Cfg::SOFTMAX_WARPS) {
      constexpr int LPR = W / 4;     // lanes per row (one 16-byte chunk each)
      constexpr int RPI = 32 / LPR;  // rows per warp iteration
      const int chunk = lane % LPR, sub = lane / LPR;
      const int x = warp >> 2;
      // a CTA of the cluster that gave up on a wait has set the status word (before the barrier): its partials are
      // incomplete, so nobody writes rows merged from them
      const bool cta_ok = *abort_flag == 0 && *reinterpret_cast<volatile int*>(p.status) == 0;
      if (Tg[x] > 0) {  // the query tile exists
        // This lane finishes one 16-byte chunk of the rows (warp & 3) * 32 + it * RPI + sub, it = 0..LPR-1.
        // Loads go to L2 (the lines were written by other SMs) and are issued in batches before their first use.
        auto row_of = [&](int it) { return (warp & 3) * 32 + it * RPI + sub; };
        float2 ml[LPR][CL];
#pragma unroll
        for (int it = 0; it < LPR; ++it)
#pragma unroll
          for (int cr = 0; cr < CL; ++cr)
            ml[it][cr] = __ldcg(reinterpret_cast<const float2*>(gml + cr * TC_ML_FLOATS) + x * TC_BM + row_of(it));
        float wgt[LPR][CL];  // weight of CTA cr's partial in row it, normalisation included
#pragma unroll
        for (int it = 0; it < LPR; ++it) {
          float m = -INFINITY;
#pragma unroll
          for (int cr = 0; cr < CL; ++cr)
            if (ml[it][cr].y > 0.f) m = fmaxf(m, ml[it][cr].x);  // a CTA whose tiles were all hidden from the row has l = 0
          float lsum = 0.f;
#pragma unroll
          for (int cr = 0; cr < CL; ++cr) {
            wgt[it][cr] = ml[it][cr].y > 0.f ? fast_exp2(ml[it][cr].x - m) : 0.f;
            lsum = fmaf(wgt[it][cr], ml[it][cr].y, lsum);
          }
          const float inv = 1.f / lsum;
#pragma unroll
          for (int cr = 0; cr < CL; ++cr) wgt[it][cr] *= inv;
          const int row = (qblk * NQ + x) * TC_BM + row_of(it);
          if (cta_ok && crank == 0 && chunk == 0 && p.lse && row < p.q_len)
            p.lse[(static_cast<int64_t>(b) * p.q_heads + h) * p.q_len + row] =
                (m + log2f(lsum)) * 0.69314718055994530942f;
        }
        constexpr int BATCH = 4;
#pragma unroll
        for (int it0 = 0; it0 < LPR; it0 += BATCH) {
          float4 v[BATCH][CL];
#pragma unroll
          for (int k = 0; k < BATCH; ++k) {
            const int r = row_of(it0 + k);
            const int off = ((crank * 2 + x) * TC_BM + r) * W + ((chunk ^ (r & 7)) << 2);
#pragma unroll
            for (int cr = 0; cr < CL; ++cr)
              v[k][cr] = __ldcg(reinterpret_cast<const float4*>(gpart + cr * TC_PART_FLOATS + off));
          }
#pragma unroll
          for (int k = 0; k < BATCH; ++k) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int cr = 0; cr < CL; ++cr) {
              const float w = wgt[it0 + k][cr];
              acc.x = fmaf(w, v[k][cr].x, acc.x);
              acc.y = fmaf(w, v[k][cr].y, acc.y);
              acc.z = fmaf(w, v[k][cr].z, acc.z);
              acc.w = fmaf(w, v[k][cr].w, acc.w);
            }
            const int row = (qblk * NQ + x) * TC_BM + row_of(it0 + k);
            if (cta_ok && row < p.q_len)
              *reinterpret_cast<float4*>(p.out + ((static_cast<int64_t>(b) * p.q_len + row) * p.q_heads + h) * TC_D +
                                         crank * W + chunk * 4) = acc;
          }
        }
      }
    }
  }

  // ---- tear-down
  tc_fence_before();
  __syncthreads();
  if (warp == Cfg::MMA_WARP) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace jup

#include "prefill_tc_frag.cuh"

namespace jup {

// ---------------------------------------------------------------- host side

static cudaError_t launch_frag(int64_t ctas, cudaStream_t st, const CUtensorMap& tq, const CUtensorMap& tk,
                               const CUtensorMap& tv, const CUtensorMap& tpk, const CUtensorMap& tpv,
                               const CUtensorMap& tck, const CUtensorMap& tcv, const TcParams& p) {
  static PerDeviceOnce done;
  if (!done.done()) {
    cudaError_t e =
        cudaFuncSetAttribute(prefill_frag_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FragCfg::SMEM_BYTES);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(prefill_frag_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    done.set();
  }
  return launch_pdl_cluster(prefill_frag_kernel, dim3(static_cast<unsigned>(ctas)), dim3(FragCfg::THREADS),
                            FragCfg::SMEM_BYTES, st, 1u, tq, tk, tv, tpk, tpv, tck, tcv, p);
}

template <int CL>
static cudaError_t launch_variant(int64_t ctas, cudaStream_t st, const CUtensorMap& tq, const CUtensorMap& tk,
                                  const CUtensorMap& tv, const CUtensorMap& tpk, const CUtensorMap& tpv,
                                  const CUtensorMap& to, const CUtensorMap& tck, const CUtensorMap& tcv,
                                  const TcParams& p) {
  using Cfg = TcCfg;
  static PerDeviceOnce done;
  if (!done.done()) {
    cudaError_t e =
        cudaFuncSetAttribute(prefill_tc_kernel<CL>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(prefill_tc_kernel<CL>, cudaFuncAttributePreferredSharedMemoryCarveout,
                               cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    done.set();
  }
  return launch_pdl_cluster(prefill_tc_kernel<CL>, dim3(static_cast<unsigned>(ctas * CL)),
                            dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, static_cast<unsigned>(CL), tq, tk, tv, tpk, tpv, to, tck,
                            tcv, p);
}

// How many clusters of CL CTAs of the cluster-mode kernel can be resident at once (0 if the query fails).
template <int CL>
static int max_resident_clusters() {
  static std::atomic<int> cache[64];  // per device: 0 = not asked yet, else answer + 1
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  const int cached = cache[dev].load(std::memory_order_acquire);
  if (cached > 0) return cached - 1;
  using Cfg = TcCfg;
  int n = 0;
  if (cudaFuncSetAttribute(prefill_tc_kernel<CL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           Cfg::SMEM_BYTES) == cudaSuccess) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(CL * 64);
    cfg.blockDim = dim3(Cfg::THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int got = 0;
    if (cudaOccupancyMaxActiveClusters(&got, prefill_tc_kernel<CL>, &cfg) == cudaSuccess) n = got;
    else (void)cudaGetLastError();
  } else {
    (void)cudaGetLastError();
  }
  cache[dev].store(n + 1, std::memory_order_release);
  return n;
}

bool prefill_tc_supported(const CacheView& c, float scale) {
  // head_dim 128, a positive finite scale, and strides a tensor map can carry (multiples of 16 bytes below 2^40;
  // the 16-byte rule is part of every cache descriptor already)
  auto encodable = [](int64_t elems) { return static_cast<uint64_t>(elems) * 2 < (1ull << 40); };
  return c.head_dim == TC_D && scale > 0.f && scale < INFINITY && encode_fn() != nullptr && encodable(c.sr) &&
         encodable(c.sh) && encodable(c.sb);
}

// c: the attention's own segment (rows [0, pos + q_len) of every sequence); prefix (nullable): the segment in front
// of it, shared by all sequences or one per sequence (prefix_batched); copy_dst (nullable): cache that receives the
// own segment's rows at copy_pos (the own segment is then the chunk's token-major K/V).
static cudaError_t launch_tc(const bf16* q, const CacheView& c, const CacheView* prefix, int prefix_len,
                             bool prefix_batched, const CacheView* copy_dst, int copy_pos, int q_heads, int q_len,
                             int pos, float scale, float* out, float* lse, int* status, void* workspace,
                             size_t workspace_bytes, cudaStream_t st, LaunchInfo& li) {
  CUtensorMap tq, tk, tv, tpk, tpv, to, tck, tcv;
  if (!encode_fn()) return cudaErrorInvalidValue;
  {  // out: [batch][q_len][q_heads][128] fp32, boxes of 128 rows x 32 columns
    const uint64_t d[4] = {TC_D, static_cast<uint64_t>(q_heads), static_cast<uint64_t>(q_len),
                           static_cast<uint64_t>(c.batch)};
    const uint64_t s[3] = {TC_D * 4ull, static_cast<uint64_t>(q_heads) * TC_D * 4ull,
                           static_cast<uint64_t>(q_len) * q_heads * TC_D * 4ull};
    const uint32_t bx[4] = {32, 1, TC_BM, 1};
    if (!make_map_f32(&to, out, d, s, bx)) return cudaErrorInvalidValue;
  }
  const uint64_t rows_valid = static_cast<uint64_t>(pos) + q_len;  // rows above are dead: TMA zero-fills them
  {
    const uint64_t d[4] = {TC_D, static_cast<uint64_t>(q_heads), static_cast<uint64_t>(q_len),
                           static_cast<uint64_t>(c.batch)};
    const uint64_t s[3] = {TC_D * 2ull, static_cast<uint64_t>(q_heads) * TC_D * 2ull,
                           static_cast<uint64_t>(q_len) * q_heads * TC_D * 2ull};
    const uint32_t bx[4] = {64, 1, TC_BM, 1};
    if (!make_map_bf16(&tq, q, d, s, bx)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t d[4] = {TC_D, rows_valid, static_cast<uint64_t>(c.kv_heads), static_cast<uint64_t>(c.batch)};
    const uint64_t s[3] = {static_cast<uint64_t>(c.sr) * 2, static_cast<uint64_t>(c.sh) * 2,
                           static_cast<uint64_t>(c.sb) * 2};
    const uint32_t bx[4] = {64, TC_BN, 1, 1};
    if (!make_map_bf16(&tk, c.k, d, s, bx) || !make_map_bf16(&tv, c.v, d, s, bx)) return cudaErrorInvalidValue;
  }
  if (prefix && prefix_len > 0) {  // rows at or beyond prefix_len are zero-filled by TMA
    const uint64_t d[4] = {TC_D, static_cast<uint64_t>(prefix_len), static_cast<uint64_t>(prefix->kv_heads),
                           static_cast<uint64_t>(prefix_batched ? prefix->batch : 1)};
    const uint64_t s[3] = {static_cast<uint64_t>(prefix->sr) * 2, static_cast<uint64_t>(prefix->sh) * 2,
                           static_cast<uint64_t>(prefix->sb) * 2};
    const uint32_t bx[4] = {64, TC_BN, 1, 1};
    if (!make_map_bf16(&tpk, prefix->k, d, s, bx) || !make_map_bf16(&tpv, prefix->v, d, s, bx)) return cudaErrorInvalidValue;
  } else {
    tpk = tk;  // never dereferenced when there is no prefix
    tpv = tv;
    prefix_len = 0;
  }
  TcParams p;
  p.q_heads = q_heads;
  p.group = q_heads / c.kv_heads;
  p.q_len = q_len;
  p.pos = pos;
  p.prefix_len = prefix_len;
  p.batch = c.batch;
  p.scale_log2 = scale * 1.4426950408889634f;
  p.prefix_batched = prefix_batched ? 1 : 0;
  p.fused_write = copy_dst ? 1 : 0;
  p.copy_pos = copy_dst ? copy_pos : 0;
  tck = tk;  // never dereferenced without a fused write
  tcv = tv;
  if (copy_dst) {  // destination rows [0, copy_pos + q_len) of every sequence's cache; stores beyond are clipped
    const uint64_t d[4] = {TC_D, static_cast<uint64_t>(copy_pos) + q_len, static_cast<uint64_t>(copy_dst->kv_heads),
                           static_cast<uint64_t>(copy_dst->batch)};
    const uint64_t s[3] = {static_cast<uint64_t>(copy_dst->sr) * 2, static_cast<uint64_t>(copy_dst->sh) * 2,
                           static_cast<uint64_t>(copy_dst->sb) * 2};
    const uint32_t bx[4] = {64, TC_BN, 1, 1};
    if (!make_map_bf16(&tck, copy_dst->k, d, s, bx) || !make_map_bf16(&tcv, copy_dst->v, d, s, bx)) return cudaErrorInvalidValue;
  }
  p.out = out;
  p.lse = lse;
  p.status = status;
  // Two query tiles per CTA when that still fills the machine (every K/V tile then serves two query tiles).  A
  // grid that leaves SMs idle is latency-bound on the walk over the KV tiles: with few pairs of query tiles and a
  // long walk, a cluster of 4 CTAs shares a pair and splits the walk; the exchange of the partials costs about
  // 10 us, so the cluster pays from about 18 KV tiles on (measured on chunk 256 x 32 heads), and only while all
  // clusters are resident at once.  Otherwise one query tile per CTA (fragment form).
  const int64_t ctas2 = static_cast<int64_t>((q_len + 255) / 256) * c.batch * q_heads;
  const int64_t ctas1 = static_cast<int64_t>((q_len + 127) / 128) * c.batch * q_heads;
  const int kv_tiles = (prefix_len + TC_BN - 1) / TC_BN + (pos + q_len + TC_BN - 1) / TC_BN;
  int cl = 1;
  if (ctas2 < li.sm_count && q_len > TC_BM) {
    // scratch for the partials behind the counter block at the head of the workspace
    auto fits = [&](int n) {
      return workspace && SCRATCH_COUNTER_BYTES + static_cast<size_t>(ctas2) * n * (TC_PART_FLOATS + TC_ML_FLOATS) * 4 <=
                              workspace_bytes;
    };
    if (ctas2 * 4 <= li.sm_count && kv_tiles >= TC_CLUSTER_MIN_TILES && fits(4) && max_resident_clusters<4>() >= ctas2)
      cl = 4;
  }
  p.scratch = cl > 1 ? reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + SCRATCH_COUNTER_BYTES) : nullptr;
  cudaError_t e;
  if (ctas2 >= li.sm_count) {
    p.q_blocks = (q_len + 255) / 256;
    e = launch_variant<1>(ctas2, st, tq, tk, tv, tpk, tpv, to, tck, tcv, p);
  } else if (cl == 4) {
    p.q_blocks = (q_len + 255) / 256;
    e = launch_variant<4>(ctas2, st, tq, tk, tv, tpk, tpv, to, tck, tcv, p);
  } else {
    p.q_blocks = (q_len + 127) / 128;
    e = launch_frag(ctas1, st, tq, tk, tv, tpk, tpv, tck, tcv, p);
  }
  li.launches += 1;
  return e;
}

cudaError_t launch_prefill_tc(const bf16* q, const CacheView& c, const CacheView* prefix, int prefix_len,
                              int q_heads, int q_len, int pos, float scale, float* out, float* lse, int* status,
                              void* workspace, size_t workspace_bytes, cudaStream_t st, LaunchInfo& li) {
  return launch_tc(q, c, prefix, prefix_len, false, nullptr, 0, q_heads, q_len, pos, scale, out, lse, status, workspace,
                   workspace_bytes, st, li);
}

cudaError_t launch_prefill_tc_fused(const bf16* q, const CacheView& c, const bf16* k_new, const bf16* v_new,
                                    int q_heads, int q_len, int pos, float scale, float* out, float* lse, int* status,
                                    void* workspace, size_t workspace_bytes, cudaStream_t st, LaunchInfo& li) {
  // own segment: the chunk itself, [batch][q_len][kv_heads][128] seen as a cache of q_len rows at position 0;
  // front segment: rows [0, pos) of each sequence's cache
  CacheView own;
  own.k = k_new;
  own.v = v_new;
  own.batch = c.batch;
  own.kv_heads = c.kv_heads;
  own.capacity = q_len;
  own.head_dim = c.head_dim;
  own.sr = static_cast<int64_t>(c.kv_heads) * c.head_dim;
  own.sh = c.head_dim;
  own.sb = static_cast<int64_t>(q_len) * own.sr;
  return launch_tc(q, own, pos > 0 ? &c : nullptr, pos, true, &c, pos, q_heads, q_len, 0, scale, out, lse, status,
                   workspace, workspace_bytes, st, li);
}

}  // namespace jup
