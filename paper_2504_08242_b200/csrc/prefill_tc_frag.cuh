// Chunked-prefill attention, one query tile of 128 rows per CTA, both softmax warpgroups on that tile
// (included by prefill_tc.cu, which holds the parameters, the tensor maps and the dispatch).
//
// TMEM: S0 | S1 | S2 | O (128 columns each).  The MMA issuer runs S(j+3) = Q K(j+3)^T right after O += P(j) V(j),
// into the buffer P(j) is read from, so the scores of a tile are complete a whole tile before its softmax starts:
// the softmax never waits for the tensor pipe, and it can fetch the next tile's scores into registers and reduce
// them to their row maxima while the exponentials of the current tile keep the special-function unit busy.  A
// tile then costs about what its exponentials cost.  The two warpgroups split the tile by rows (warp w owns the 16
// rows 32 (w mod 4) + 16 (w / 4) ..., in the 16x256b fragment layout, see tc_softmax.cuh), so every warp scheduler
// works on every tile; a softmax thread holds two tiles' fragments (the register file is re-divided).
//   warps 0-7 : softmax;  warp 8: loader (TMA);  warp 9: MMA issuer;  warp 10: watcher;  warp 11: idle
// The issuer thread is blocked while the tensor pipe works through its queue, so whatever else it executes adds to
// the pipe's idle time: it tests no barrier and commits once per tile.  The watcher thread waits for each step's
// conditions in the issuer's program order and counts the cleared steps in shared memory (the issuer reads that
// word).  The loader needs no "slot empty" barriers: S(i) complete means S = Q K(i)^T has read K(i)'s slot and
// O += P V of tile i - 3, issued before it, has read V(i-3)'s slot.
#pragma once

namespace jup {

struct FragCfg {
  static constexpr int STAGES = 3;  // K slots = V slots = S buffers
  static constexpr int SOFTMAX_WARPS = 8, LOADER_WARP = 8, MMA_WARP = 9, WATCH_WARP = 10;
  static constexpr int THREADS = 384;
  static constexpr int REGS_SOFTMAX = 216, REGS_OTHER = 72;  // 2 x 128 x 216 + 128 x 72 = 384 x 168
  static constexpr int O_COL0 = 384;
  static constexpr int SMEM_Q = 0;
  static constexpr int SMEM_K = TC_TILE_BYTES;
  static constexpr int SMEM_V = SMEM_K + STAGES * TC_TILE_BYTES;
  static constexpr int SMEM_BAR = SMEM_V + STAGES * TC_TILE_BYTES;
  static constexpr int SMEM_BYTES = SMEM_BAR + 256 + 1024;  // + slack for 1024-byte alignment
  static_assert(SMEM_BYTES <= 227 * 1024, "shared memory per CTA");
};
enum {
  FB_Q_FULL = 0,
  FB_K_FULL = 1,    // [3] slot j % 3, phase j / 3
  FB_V_FULL = 4,    // [3]
  FB_S_FULL = 7,    // [3] buffer j % 3, phase j / 3
  FB_P_FULL = 10,   // [3] one arrival per softmax warp
  FB_O_READY = 13,  // [3] one barrier (a single phase) for each of the last (up to) three tiles' O += P V: a
                    // thread may come to them long after they completed, which one barrier's parity could not tell
  FB_DRAIN = 16,
  FB_COUNT = 17
};

__global__ void __launch_bounds__(FragCfg::THREADS, 1)
prefill_frag_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_pk,
                    const __grid_constant__ CUtensorMap tm_pv, const __grid_constant__ CUtensorMap tm_ck,
                    const __grid_constant__ CUtensorMap tm_cv, TcParams p) {
  using Cfg = FragCfg;
  constexpr int STAGES = Cfg::STAGES;
  extern __shared__ unsigned char smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t sQ = smem_base + Cfg::SMEM_Q, sK = smem_base + Cfg::SMEM_K, sV = smem_base + Cfg::SMEM_V;
  const uint32_t sBar = smem_base + Cfg::SMEM_BAR;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + Cfg::SMEM_BAR + 8 * FB_COUNT);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + Cfg::SMEM_BAR + 8 * FB_COUNT + 8);
  const uint32_t go_count = sBar + 8u * FB_COUNT + 16u;  // steps the watcher has cleared for the issuer
  static_assert(8 * FB_COUNT + 24 <= 256, "barrier block");
  auto bar = [&](int i) { return sBar + 8u * i; };
  // barrier (of a family of three) and parity of tile j
  auto bar3 = [&](int family, int j) { return sBar + 8u * (family + j % STAGES); };
  auto par3 = [](int j) { return static_cast<uint32_t>(j / STAGES) & 1u; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // ---- work assignment: heaviest query tiles first
  const int nbh = p.batch * p.q_heads;
  const int bh = blockIdx.x % nbh;
  const int qblk = p.q_blocks - 1 - blockIdx.x / nbh;
  const int b = bh / p.q_heads, h = bh % p.q_heads, hk = h / p.group;
  // KV tiles 0..Tp-1 come from the front segment (every row sees them, no causal limit), the rest from the own one
  const int Tp = (p.prefix_len + TC_BN - 1) / TC_BN;
  const int T = Tp + (p.pos + min(p.q_len, (qblk + 1) * TC_BM) + TC_BN - 1) / TC_BN;  // >= 1
  // O += P V of tile j is followed by S(j+3), whose barrier then also says that the accumulator holds tile j; the
  // last tiles have no S(j+3) and complete one of the accumulator's own barriers instead, the first for tile o0
  const int o0 = max(T - STAGES, 0);

  if (threadIdx.x == 0) {
    for (int i = 0; i < FB_COUNT; ++i)
      mbar_init(bar(i), (i >= FB_P_FULL && i < FB_P_FULL + STAGES) ? static_cast<uint32_t>(Cfg::SOFTMAX_WARPS) : 1u);
    *abort_flag = 0;
    *reinterpret_cast<volatile int*>(smem_gen + Cfg::SMEM_BAR + 8 * FB_COUNT + 16) = 0;
    mbar_fence_init();
  }
  if (warp == Cfg::MMA_WARP) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish();
  } else if (warp == Cfg::LOADER_WARP && lane == 0) {
    tma_prefetch_desc(&tm_q);
    tma_prefetch_desc(&tm_k);
    tma_prefetch_desc(&tm_v);
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

  if (warp == Cfg::LOADER_WARP) {
    // =============================================================== loader
    reg_dec<Cfg::REGS_OTHER>();
    if (lane == 0) {
      const int r0 = qblk * TC_BM;
      mbar_expect_tx(bar(FB_Q_FULL), TC_TILE_BYTES);
      tma_load_4d(sQ, &tm_q, bar(FB_Q_FULL), 0, h, r0, b);
      tma_load_4d(sQ + TC_PANEL_BYTES, &tm_q, bar(FB_Q_FULL), 64, h, r0, b);
      bool ok = true;
      int k_issued = 0, v_issued = 0;
      auto load = [&](bool is_v, int j) {
        const int s = j % STAGES;
        const uint32_t full = bar3(is_v ? FB_V_FULL : FB_K_FULL, j);
        const uint32_t dst = (is_v ? sV : sK) + s * TC_TILE_BYTES;
        const CUtensorMap* m = j < Tp ? (is_v ? &tm_pv : &tm_pk) : (is_v ? &tm_v : &tm_k);
        const int krow = (j < Tp ? j : j - Tp) * TC_BN, kb = (j < Tp && !p.prefix_batched) ? 0 : b;
        mbar_expect_tx(full, TC_TILE_BYTES);
        tma_load_4d(dst, m, full, 0, krow, hk, kb);
        tma_load_4d(dst + TC_PANEL_BYTES, m, full, 64, krow, hk, kb);
        if (is_v) v_issued = j + 1;
        else k_issued = j + 1;
      };
      // Fused KVCache write: the chunk's own K/V tile that holds this CTA's query rows goes from its slots to the
      // cache with tiled stores once it has landed, before the slot is refilled (CTAs of each group's first query
      // head only); rows beyond copy_pos + q_len are clipped by the tensor maps.
      const int j_own = (p.fused_write != 0 && h % p.group == 0) ? Tp + qblk : -1;
      auto store_own = [&](bool is_v) {
        ok = ok && mbar_wait(bar3(is_v ? FB_V_FULL : FB_K_FULL, j_own), par3(j_own), abort_flag, p.status);
        if (!ok) return;
        const uint32_t src = (is_v ? sV : sK) + (j_own % STAGES) * TC_TILE_BYTES;
        const CUtensorMap* m = is_v ? &tm_cv : &tm_ck;
        const int row = p.copy_pos + qblk * TC_BN;
        tma_store_4d(m, src, 0, row, hk, b);
        tma_store_4d(m, src + TC_PANEL_BYTES, 64, row, hk, b);
        tma_store_commit();
        tma_store_wait_read();
      };
      for (int j = 0; j < STAGES && j < T; ++j) {
        load(false, j);
        load(true, j);
      }
      bool v_stored = false;
      for (int i = 0; i < T && ok; ++i) {
        ok = mbar_wait(bar3(FB_S_FULL, i), par3(i), abort_flag, p.status);
        if (!ok) break;
        if (j_own >= 0 && i == j_own) store_own(false);
        if (j_own >= 0 && i - STAGES == j_own) {
          store_own(true);
          v_stored = true;
        }
        if (!ok) break;
        if (i + STAGES < T) load(false, i + STAGES);  // K(i)'s slot
        if (i >= STAGES) load(true, i);               // V(i-3)'s slot
      }
      if (ok && j_own >= 0 && !v_stored) store_own(true);
      if (*abort_flag) {
        // wait (bounded) until every copy this thread started has landed before shared memory is released
        int dummy = 0;
        volatile int* none = &dummy;
        for (int j = max(0, k_issued - STAGES); j < k_issued; ++j) mbar_wait(bar3(FB_K_FULL, j), par3(j), none, nullptr);
        for (int j = max(0, v_issued - STAGES); j < v_issued; ++j) mbar_wait(bar3(FB_V_FULL, j), par3(j), none, nullptr);
        mbar_wait(bar(FB_Q_FULL), 0, none, nullptr);
      }
    }
    __syncwarp();
  } else if (warp == Cfg::MMA_WARP) {
    // =============================================================== MMA issuer
    // Steps (each cleared by the watcher):  S(0), S(1), S(2);  then per tile j:  O += P(j) V(j),  S(j+3).
    reg_dec<Cfg::REGS_OTHER>();
    if (lane == 0) {
      constexpr uint32_t idesc_qk = tc_idesc_bf16(TC_BM, TC_BN, false, false);
      constexpr uint32_t idesc_pv = tc_idesc_bf16(TC_BM, TC_D, false, true);
      const uint32_t q_lo = tc_desc_lo(sQ, 16), k_lo0 = tc_desc_lo(sK, 16), v_lo0 = tc_desc_lo(sV, TC_PANEL_BYTES);
      const uint32_t o_col = tmem + Cfg::O_COL0;
      // slot of K and V and S buffer are all j mod 3
      auto issue_qk = [&](int s) {  // S[s] = Q K[s]^T
        const uint32_t k_lo = k_lo0 + s * (TC_TILE_BYTES >> 4);
        const uint32_t d = tmem + s * 128;
#pragma unroll
        for (int ks = 0; ks < TC_D / 16; ++ks) {
          const uint32_t off = ((ks >> 2) * TC_PANEL_BYTES + (ks & 3) * 32) >> 4;
          tc_mma_ss_lo(d, q_lo + off, k_lo + off, idesc_qk, ks > 0);
        }
      };
      auto issue_pv = [&](int s, bool first) {  // O (+)= P[s] V[s]
        const uint32_t v_lo = v_lo0 + s * (TC_TILE_BYTES >> 4);
        const uint32_t a = tmem + s * 128;
#pragma unroll
        for (int ks = 0; ks < TC_BN / 16; ++ks)
          tc_mma_ts_lo(o_col, a + ks * 8, v_lo + ks * (2048 >> 4), idesc_pv, (!first || ks > 0));
      };
      int cleared = 0, step = 0;  // steps the watcher is known to have cleared / steps taken
      bool ok = true;
      auto next_step = [&] {
        ++step;
        if (cleared < step) {
          cleared = count_spin_wait(go_count, step, abort_flag, p.status);
          ok = cleared >= 0;
        }
        tc_fence_after();
        return ok;
      };
      for (int j = 0; j < STAGES && j < T && ok; ++j) {
        if (!next_step()) break;
        issue_qk(j);
        tc_commit(bar(FB_S_FULL + j));
      }
      int s = 0;
      for (int j = 0; j < T && ok; ++j) {
        if (!next_step()) break;
        issue_pv(s, j == 0);
        if (j + STAGES < T) {
          issue_qk(s);
          tc_commit(bar(FB_S_FULL + s));
        } else {
          tc_commit(bar(FB_O_READY + j - o0));
        }
        s = s + 1 == STAGES ? 0 : s + 1;
      }
      if (!ok) {  // make sure no MMA of this thread is still running before TMEM and smem go away
        int dummy = 0;
        tc_commit(bar(FB_DRAIN));
        mbar_wait(bar(FB_DRAIN), 0, &dummy, nullptr);
      }
    }
    __syncwarp();
  } else if (warp == Cfg::WATCH_WARP) {
    // =============================================================== watcher (see the MMA issuer)
    reg_dec<Cfg::REGS_OTHER>();
    if (lane == 0) {
      bool ok = mbar_wait(bar(FB_Q_FULL), 0, abort_flag, p.status);
      int step = 0;
      auto landed = [&](int family, int j) { return mbar_wait(bar3(family, j), par3(j), abort_flag, p.status); };
      for (int j = 0; j < STAGES && j < T && ok; ++j) {
        ok = landed(FB_K_FULL, j);
        if (ok) count_publish(go_count, ++step);
      }
      for (int j = 0; j < T && ok; ++j) {
        ok = landed(FB_V_FULL, j);
        if (ok && j + STAGES < T) ok = landed(FB_K_FULL, j + STAGES);
        ok = ok && mbar_spin_wait(bar3(FB_P_FULL, j), par3(j), abort_flag, p.status);
        if (!ok) break;
        count_publish(go_count, ++step);
      }
    }
    __syncwarp();
  } else if (warp < Cfg::SOFTMAX_WARPS) {
    // =============================================================== softmax: 16 rows per warp
    reg_inc<Cfg::REGS_SOFTMAX>();
    const int lane0 = (warp & 3) * 32 + (warp >> 2) * 16;  // first TMEM lane (row of the tile) of this warp
    const int col0 = 2 * (lane & 3);
    const uint32_t taddr = tmem + (static_cast<uint32_t>(lane0) << 16);
    const uint32_t tO = taddr + Cfg::O_COL0;
    int row[2], lim[2];  // row inside the chunk and its causal limit (keys j < lim are visible)
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      row[e] = qblk * TC_BM + lane0 + (lane >> 2) + 8 * e;
      lim[e] = p.pos + min(row[e], p.q_len - 1) + 1;
    }
    const float c = p.scale_log2;
    float m_ref[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
    float mxs[2];
    bool ok = true;
    // the accumulator holds tile j - 1 (needed before its rows are rescaled at tile j)
    auto wait_o_before = [&](int j) {
      if (j + 2 < T) return mbar_wait(bar3(FB_S_FULL, j + 2), par3(j + 2), abort_flag, p.status);
      return mbar_wait(bar(FB_O_READY + j - 1 - o0), 0, abort_flag, p.status);
    };
    // Scores of tile j into fragments (asynchronous: the registers may only be used after the load was waited for).
    auto fetch = [&](int j, uint32_t (&sv)[64]) {
      ok = mbar_spin_wait(bar3(FB_S_FULL, j), par3(j), abort_flag, p.status);
      if (!ok) return;
      tc_fence_after();
      tmem_ld_16x256b_x16(taddr + (j % STAGES) * 128, sv);
    };
    // Columns >= nvalid of a row are hidden: the end of the front segment in its last tile, the causal limit afterwards.
    int nvalid[2];
    auto tile_masked = [&](int j) {  // warp-uniform; fills nvalid
#pragma unroll
      for (int e = 0; e < 2; ++e) nvalid[e] = j < Tp ? p.prefix_len - j * TC_BN : lim[e] - (j - Tp) * TC_BN;
      return __any_sync(0xffffffffu, nvalid[0] < TC_BN || nvalid[1] < TC_BN) != 0;
    };
    auto apply_mask = [&](uint32_t (&sv)[64]) {
#pragma unroll
      for (int k = 0; k < 16; ++k)
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (8 * k + col0 + (i & 1) >= nvalid[i >> 1]) sv[4 * k + i] = 0xff800000u;  // -inf
    };
    // One tile: cur holds its masked scores and mxs its maxima; nxt is the next tile's fetch in flight, whose maxima
    // are worked out between this tile's exponentials; afterwards the fetch of the tile after that goes into cur.
    auto tile = [&](int j, uint32_t (&cur)[64], uint32_t (&nxt)[64]) {
      if (!frag_decide(mxs, m_ref, l, tO, j, [&] { return wait_o_before(j); })) {
        ok = false;
        return;
      }
      const bool next_masked = j + 1 < T && tile_masked(j + 1);
      float mxs_next[2];
      frag_exp_store_max(cur, taddr + (j % STAGES) * 128, c, m_ref, l, nxt, next_masked, [&] { apply_mask(nxt); }, mxs_next);
      mxs[0] = mxs_next[0];
      mxs[1] = mxs_next[1];
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar3(FB_P_FULL, j));
      if (j + 2 < T) fetch(j + 2, cur);
    };
    uint32_t fa[64], fb[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) fb[i] = 0u;  // read (and ignored) as "next tile" when there is none
    fetch(0, fa);
    if (ok) {
      tc_wait_ld_into(fa);
      const bool masked0 = tile_masked(0);
      frag_mask_max(fa, masked0, [&](int e, int col) { return col < nvalid[e]; }, col0, c, mxs);
      if (T > 1) fetch(1, fb);
    }
    for (int j = 0; j < T && ok; j += 2) {
      tile(j, fa, fb);
      if (j + 1 < T && ok) tile(j + 1, fb, fa);
    }
    tc_wait_ld();  // (no fetch is left in flight; the registers are dead)
    pdl_launch_dependents();  // the next kernel of the stream may start its own set-up now
    ok = ok && mbar_wait(bar(FB_O_READY + T - 1 - o0), 0, abort_flag, p.status);  // the accumulator is final
    tc_fence_after();
    // ---- output: O / l straight from the fragments (a row's four threads write 32 contiguous bytes per repeat)
    float inv[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      l[e] += __shfl_xor_sync(0xffffffffu, l[e], 1);
      l[e] += __shfl_xor_sync(0xffffffffu, l[e], 2);
      inv[e] = 1.f / l[e];
    }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      uint32_t o[32];
      tmem_ld_16x256b_x8(tO + hh * 64, o);
      tc_wait_ld();
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        if (!ok || row[e] >= p.q_len) continue;
        float* dst = p.out + ((static_cast<int64_t>(b) * p.q_len + row[e]) * p.q_heads + h) * TC_D + hh * 64 + col0;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          *reinterpret_cast<float2*>(dst + 8 * k) =
              make_float2(__uint_as_float(o[4 * k + 2 * e]) * inv[e], __uint_as_float(o[4 * k + 2 * e + 1]) * inv[e]);
      }
    }
    if (ok && p.lse && (lane & 3) == 0) {
#pragma unroll
      for (int e = 0; e < 2; ++e)
        if (row[e] < p.q_len)
          p.lse[(static_cast<int64_t>(b) * p.q_heads + h) * p.q_len + row[e]] =
              (m_ref[e] + log2f(l[e])) * 0.69314718055994530942f;
    }
  } else {
    reg_dec<Cfg::REGS_OTHER>();  // the idle warp of the third warpgroup: the re-division is a warpgroup's decision
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
