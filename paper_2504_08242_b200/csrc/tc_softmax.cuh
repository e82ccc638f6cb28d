// The online-softmax steps of the tcgen05 attention kernels, three forms of the same arithmetic -- P = exp2(s c - m)
// with fp32-pair instructions, written back over S in TMEM as bf16 pairs (P column k holds keys 2k and 2k + 1, so the
// writes stay behind the reads), a lazy reference maximum m that only moves when the tile's maximum outgrew it by more
// than 2^8 (then the row sum and the accumulator O are scaled by exp2(m_old - m_new); with well-behaved scores that
// happens in a row's first tile and almost never again):
//   softmax_tile_step : a thread per row, the row's 128 scores walked once in four chunks of 32 columns with the next
//                       chunk in flight (about 160 registers; the branch kernel)
//   softmax_tile_row  : a thread per row holding the whole row (about 200 registers), P released in two parts (the
//                       two-tile prefill kernel)
//   frag_*            : 16 rows per warp in the 16x256b fragment layout, in pieces that a kernel interleaves across
//                       consecutive tiles (the one-tile prefill kernel)
#pragma once
#include "tc_common.cuh"

namespace jup {

constexpr float TC_RESCALE_THRESHOLD = 8.f;  // log2 units

// Visibility of the tile's columns to this thread's row (only consulted on tiles flagged as masked).
struct ColumnLimit {  // columns [0, nvalid) are visible
  int nvalid;
  __device__ __forceinline__ bool operator()(int col) const { return col < nvalid; }
};
struct ColumnBits {  // bit (col & 31) of w[col >> 5] set: visible
  uint32_t w[4];
  __device__ __forceinline__ bool operator()(int col) const { return (w[col >> 5] >> (col & 31)) & 1u; }
};

__device__ __forceinline__ uint32_t scale_bf16_pair(uint32_t pair, float a) {
  const float lo = __uint_as_float(pair << 16), hi = __uint_as_float(pair & 0xffff0000u);
  return pack_bf16(lo * a, hi * a);
}

// tS / tO: TMEM addresses (lane base included) of the row's 128 scores and of its 128 accumulator columns.
// j: number of tiles this stream has processed before (0: O holds nothing yet).
// masked: warp-uniform; when false every column is visible and `allow` is not consulted.
// PARTIAL: the stream may meet rows that see none of a tile (their reference maximum stays -inf and P is 0);
// otherwise every row sees column 0 of its first tile.
// wait_o(): waits until O(j-1) is complete (called exactly once when j > 0); returns false if the wait gave up,
// and then so does this function.  On return P is complete in TMEM (tcgen05.wait::st done); the caller fences
// and signals the MMA issuer.
template <bool PARTIAL, class Allow, class WaitO>
__device__ __forceinline__ bool softmax_tile_step(uint32_t tS, uint32_t tO, int j, bool masked, const Allow& allow,
                                                  float c, float& m_ref, float& l, WaitO&& wait_o) {
  const uint64_t c2 = pack2(c, c);
  uint64_t lacc[4];  // this tile's row sum, four chains
#pragma unroll
  for (int k = 0; k < 4; ++k) lacc[k] = pack2(0.f, 0.f);
  float alpha_total = 1.f;  // what the sum and the accumulator of the tiles before this one must be scaled by
  bool moved = false;       // warp-uniform: some row's reference moved during this tile
  uint32_t sb[2][32];
  tmem_ld32(tS, sb[0]);
#pragma unroll
  for (int q4 = 0; q4 < 4; ++q4) {
    tc_wait_ld();
    if (q4 < 3) tmem_ld32(tS + (q4 + 1) * 32, sb[(q4 + 1) & 1]);
    uint32_t(&sv)[32] = sb[q4 & 1];
    if (masked) {
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (!allow(q4 * 32 + i)) sv[i] = 0xff800000u;  // -inf
    }
    // ---- chunk maximum (eight chains of 3-input max)
    float a[8];
#pragma unroll
    for (int k = 0; k < 8; ++k)
      a[k] = fmax3(__uint_as_float(sv[4 * k]), __uint_as_float(sv[4 * k + 1]), __uint_as_float(sv[4 * k + 2]));
    const float mx = fmax3(fmax3(fmax3(a[0], a[1], a[2]), fmax3(a[3], a[4], a[5]), fmaxf(a[6], a[7])),
                           fmax3(__uint_as_float(sv[3]), __uint_as_float(sv[7]), __uint_as_float(sv[11])),
                           fmax3(fmax3(__uint_as_float(sv[15]), __uint_as_float(sv[19]), __uint_as_float(sv[23])),
                                 __uint_as_float(sv[27]), __uint_as_float(sv[31])));
    const float mxs = mx * c;
    // lazy reference: it only moves when the maximum outgrew it by 2^8 (a row that has seen nothing keeps -inf,
    // and its first visible score moves it because -inf + 8 is still -inf)
    const bool grow = mxs > m_ref + TC_RESCALE_THRESHOLD;
    if (__any_sync(0xffffffffu, grow)) {
      const float alpha = grow ? fast_exp2(m_ref - mxs) : 1.f;
      const uint64_t al2 = pack2(alpha, alpha);
#pragma unroll
      for (int k = 0; k < 4; ++k) lacc[k] = mul2(lacc[k], al2);
      if (q4 > 0) {  // the P chunks of this tile written so far were relative to the old reference
        tc_wait_st();
#pragma unroll
        for (int qq = 0; qq < 3; ++qq) {
          if (qq >= q4) break;
          uint32_t pk[16];
          tmem_ld16(tS + qq * 16, pk);
          tc_wait_ld();  // (also completes the load of the next chunk, which is consumed later anyway)
#pragma unroll
          for (int i = 0; i < 16; ++i) pk[i] = scale_bf16_pair(pk[i], alpha);
          tmem_st16(tS + qq * 16, pk);
        }
      }
      alpha_total *= alpha;
      moved = true;
      if (grow) m_ref = mxs;
    }
    // ---- P
    const float nm = (PARTIAL && m_ref == -INFINITY) ? 0.f : -m_ref;
    const uint64_t nm2 = pack2(nm, nm);
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint64_t x = fma2(pack2(__uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1])), c2, nm2);
      float x0, x1;
      unpack2(x, x0, x1);
      const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
      lacc[i & 3] = add2(lacc[i & 3], pack2(p0, p1));
      pk[i] = pack_bf16(p0, p1);
    }
    tmem_st16(tS + q4 * 16, pk);
  }
  float l_tile;
  {
    float a0, a1, b0, b1;
    unpack2(add2(lacc[0], lacc[1]), a0, a1);
    unpack2(add2(lacc[2], lacc[3]), b0, b1);
    l_tile = (a0 + a1) + (b0 + b1);
  }
  bool o_waited = false;
  if (moved) {
    l *= alpha_total;
    if (j > 0) {  // O(j-1) must be complete before it is rescaled
      if (!wait_o()) return false;
      o_waited = true;
      tc_fence_after();
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t o[32];
        tmem_ld32(tO + q4 * 32, o);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha_total);
        tmem_st32(tO + q4 * 32, o);
      }
    }
  }
  l += l_tile;
  tc_wait_st();
  // every phase of the O-complete barrier is waited on exactly once, in order, so a parity never aliases;
  // PV(j) queues behind PV(j-1) in the tensor pipe anyway, so this costs no overlap
  if (j > 0 && !o_waited && !wait_o()) return false;
  return true;
}

// The same step with the whole score row in registers (needs about 200 registers per thread): one load of the 128
// scores, the row maximum, at most one move of the reference per tile (decided before any P is written, so no P
// chunk is ever corrected), then P in four chunks of 32 columns.  After the third chunk is in TMEM (tcgen05.wait::st
// done) release_early() runs: the caller signals the MMA issuer, which starts O += P V on the first 96 keys while
// this thread still computes the last 32.  wait_o() is only called when the accumulator has to be rescaled
// (j > 0); it waits until O(j-1) is complete and returns false if the wait gave up, and then so does this function.
// On return P is complete in TMEM; the caller fences and signals the second half.
template <bool PARTIAL, class Allow, class WaitO, class Release>
__device__ __forceinline__ bool softmax_tile_row(uint32_t tS, uint32_t tO, int j, bool masked, const Allow& allow, float c,
                                                 float& m_ref, float& l, WaitO&& wait_o, Release&& release_early) {
  uint32_t sv[128];
#pragma unroll
  for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(tS + q4 * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[q4 * 32]));
  tc_wait_ld();
  if (masked) {
#pragma unroll
    for (int i = 0; i < 128; ++i)
      if (!allow(i)) sv[i] = 0xff800000u;  // -inf
  }
  // ---- row maximum: 3-input max, 32 + 8 + 8 + 3 + 3 + 1 operations in chains of depth 5
  float mx;
  {
    float a[32];
#pragma unroll
    for (int k = 0; k < 32; ++k)
      a[k] = fmax3(__uint_as_float(sv[4 * k]), __uint_as_float(sv[4 * k + 1]), __uint_as_float(sv[4 * k + 2]));
    float b[8], d[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      b[k] = fmax3(fmax3(a[4 * k], a[4 * k + 1], a[4 * k + 2]), a[4 * k + 3], __uint_as_float(sv[16 * k + 3]));
      d[k] = fmax3(__uint_as_float(sv[16 * k + 7]), __uint_as_float(sv[16 * k + 11]), __uint_as_float(sv[16 * k + 15]));
    }
    mx = fmaxf(fmax3(fmax3(b[0], b[1], b[2]), fmax3(b[3], b[4], b[5]), fmaxf(b[6], b[7])),
               fmax3(fmax3(d[0], d[1], d[2]), fmax3(d[3], d[4], d[5]), fmaxf(d[6], d[7])));
  }
  const float mxs = mx * c;
  // lazy reference: it only moves when the maximum outgrew it by 2^8 (a row that has seen nothing keeps -inf,
  // and its first visible score moves it because -inf + 8 is still -inf)
  const bool grow = mxs > m_ref + TC_RESCALE_THRESHOLD;
  if (__any_sync(0xffffffffu, grow)) {
    const float alpha = grow ? fast_exp2(m_ref - mxs) : 1.f;
    l *= alpha;
    if (grow) m_ref = mxs;
    if (j > 0) {  // O(j-1) must be complete before it is rescaled
      if (!wait_o()) return false;
      tc_fence_after();
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t o[32];
        tmem_ld32(tO + q4 * 32, o);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
        tmem_st32(tO + q4 * 32, o);
      }
    }
  }
  // ---- P
  const float nm = (PARTIAL && m_ref == -INFINITY) ? 0.f : -m_ref;
  const uint64_t nm2 = pack2(nm, nm), c2 = pack2(c, c);
  uint64_t lacc[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) lacc[k] = pack2(0.f, 0.f);
#pragma unroll
  for (int q4 = 0; q4 < 4; ++q4) {
    uint32_t pk[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const uint64_t x =
          fma2(pack2(__uint_as_float(sv[q4 * 32 + 2 * i]), __uint_as_float(sv[q4 * 32 + 2 * i + 1])), c2, nm2);
      float x0, x1;
      unpack2(x, x0, x1);
      const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
      lacc[i & 3] = add2(lacc[i & 3], pack2(p0, p1));
      pk[i] = pack_bf16(p0, p1);
    }
    tmem_st16(tS + q4 * 16, pk);
    if (q4 == 2) {
      tc_wait_st();
      release_early();
    }
  }
  {
    float a0, a1, b0, b1;
    unpack2(add2(lacc[0], lacc[1]), a0, a1);
    unpack2(add2(lacc[2], lacc[3]), b0, b1);
    l += (a0 + a1) + (b0 + b1);
  }
  tc_wait_st();
  return true;
}

// ---------------------------------------------------------------- fragment form
// A warp owns 16 query rows of the tile (TMEM lanes lane0 .. lane0 + 15, tS / tO carry that lane) and holds their
// 128 scores in the 16x256b layout: thread t has rows A = t/4 and B = 8 + t/4, columns 8k + 2 (t mod 4) + {0, 1},
// k = 0..15 -- 64 scores per thread, half of what a thread-per-row layout holds, so two warpgroups can share one
// tile (each taking 16 of every 32 rows) and a tile's softmax takes half as long.  Row maxima are completed over
// the four threads of a row with two shuffles; the reference m_ref[e] is the same in the four threads, l[e] is a
// per-thread partial sum (added up over the quad after the walk).  Otherwise as softmax_tile_row: lazy reference,
// at most one move per tile, P written as bf16 pairs over the S columns, released in two parts.
// allow(e, col): row e (0: A, 1: B) sees column col; only consulted when masked (warp-uniform).
__device__ __forceinline__ float max32_strided(const uint32_t (&sv)[64], int e) {
  // the 32 values of row e: sv[4k + 2e], sv[4k + 2e + 1]
  float a[11];
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const int v0 = 3 * i, v1 = 3 * i + 1, v2 = 3 * i + 2;  // value indices 0..31 -> register 4 (v / 2) + 2 e + (v & 1)
    a[i] = fmax3(__uint_as_float(sv[4 * (v0 >> 1) + 2 * e + (v0 & 1)]), __uint_as_float(sv[4 * (v1 >> 1) + 2 * e + (v1 & 1)]),
                 __uint_as_float(sv[4 * (v2 >> 1) + 2 * e + (v2 & 1)]));
  }
  a[10] = fmaxf(__uint_as_float(sv[4 * 15 + 2 * e]), __uint_as_float(sv[4 * 15 + 2 * e + 1]));
  const float b0 = fmax3(a[0], a[1], a[2]), b1 = fmax3(a[3], a[4], a[5]), b2 = fmax3(a[6], a[7], a[8]);
  return fmax3(fmax3(b0, b1, b2), a[9], a[10]);
}

// The step in pieces, so that a kernel can run the pieces of consecutive tiles against each other (scores of tile
// j + 1 loaded and reduced to their row maxima while the exponentials of tile j keep the special-function unit busy).

// Row maxima (times c, over the four threads of each row) of a tile held in fragments; masks hidden columns first.
template <class Allow>
__device__ __forceinline__ void frag_mask_max(uint32_t (&sv)[64], bool masked, const Allow& allow, int col0, float c,
                                              float (&mxs)[2]) {
  if (masked) {
#pragma unroll
    for (int k = 0; k < 16; ++k)
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (!allow(i >> 1, 8 * k + col0 + (i & 1))) sv[4 * k + i] = 0xff800000u;  // -inf
  }
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    float mx = max32_strided(sv, e);
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    mxs[e] = mx * c;
  }
}

// Lazy reference: moves m_ref[e] to the tile's maximum when that outgrew it by 2^8 and scales l and, from the second
// tile on, the accumulator rows (wait_o(): bounded wait until O holds the tiles before this one; false: gave up).
template <class WaitO>
__device__ __forceinline__ bool frag_decide(const float (&mxs)[2], float (&m_ref)[2], float (&l)[2], uint32_t tO, int j,
                                            WaitO&& wait_o) {
  bool grow[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) grow[e] = mxs[e] > m_ref[e] + TC_RESCALE_THRESHOLD;
  if (__any_sync(0xffffffffu, grow[0] || grow[1])) {
    float alpha[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      alpha[e] = grow[e] ? fast_exp2(m_ref[e] - mxs[e]) : 1.f;
      l[e] *= alpha[e];
      if (grow[e]) m_ref[e] = mxs[e];
    }
    if (j > 0) {
      if (!wait_o()) return false;
      tc_fence_after();
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint32_t o[32];
        tmem_ld_16x256b_x8(tO + hh * 64, o);
        tc_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha[(i >> 1) & 1]);
        tmem_st_16x256b_x8(tO + hh * 64, o);
      }
    }
  }
  return true;
}

// Which of a tile's 32 column pairs per thread (step k, row e) take their exponentials on the FMA pipe: a quarter
// (more brought nothing: the loop is bound by dependent-issue latency, not by the special-function unit alone).
__device__ __forceinline__ constexpr bool frag_exp_on_fma(int k, int e) { return e == 1 && (k & 1) != 0; }

// P = exp2(s c - m_ref) of a tile held in fragments, as bf16 pairs over the first 64 columns of its S buffer, row
// sums into l (the stores are issued, not waited for), with the next tile's row maxima worked in: nxt is a fragment
// load in flight (or stale registers when there
// is no next tile; the result is then unused).  It is waited for after the fourth of the sixteen steps, masked if
// need be (mask_next(), warp-uniform and rare), and its 2 x 32 values are folded into running maxima a few per step,
// so that their arithmetic issues in the gaps of the exponentials instead of after them.  mxs_next: maxima times c.
template <class MaskNext>
__device__ __forceinline__ void frag_exp_store_max(const uint32_t (&sv)[64], uint32_t tS, float c, const float (&m_ref)[2],
                                                   float (&l)[2], uint32_t (&nxt)[64], bool next_masked,
                                                   MaskNext&& mask_next, float (&mxs_next)[2]) {
  uint64_t nm2[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const float nm = m_ref[e] == -INFINITY ? 0.f : -m_ref[e];
    nm2[e] = pack2(nm, nm);
  }
  const uint64_t c2 = pack2(c, c);
  uint64_t lacc[2][2];
#pragma unroll
  for (int e = 0; e < 2; ++e) lacc[e][0] = lacc[e][1] = pack2(0.f, 0.f);
  float ma[2][2] = {{-INFINITY, -INFINITY}, {-INFINITY, -INFINITY}};  // running maxima of the next tile, two chains per row
  uint32_t w[32];  // P: w[2k + e] = keys 8k + col0 + {0, 1} of row e
#pragma unroll
  for (int k = 0; k < 16; ++k) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const uint64_t x =
          fma2(pack2(__uint_as_float(sv[4 * k + 2 * e]), __uint_as_float(sv[4 * k + 2 * e + 1])), c2, nm2[e]);
      float p0, p1;
      if (frag_exp_on_fma(k, e)) {
        unpack2(exp2_poly_pair(x), p0, p1);
      } else {
        float x0, x1;
        unpack2(x, x0, x1);
        p0 = fast_exp2(x0);
        p1 = fast_exp2(x1);
      }
      lacc[e][k & 1] = add2(lacc[e][k & 1], pack2(p0, p1));
      w[2 * k + e] = pack_bf16(p0, p1);
    }
    if (k == 3) {
      tc_wait_ld_into(nxt);
      if (next_masked) mask_next();
    }
    if (k >= 4 && k < 12) {  // two of the next tile's sixteen column blocks per step
#pragma unroll
      for (int kk = 2 * (k - 4); kk < 2 * (k - 4) + 2; ++kk)
#pragma unroll
        for (int e = 0; e < 2; ++e)
          ma[e][kk & 1] = fmax3(ma[e][kk & 1], __uint_as_float(nxt[4 * kk + 2 * e]), __uint_as_float(nxt[4 * kk + 2 * e + 1]));
    }
    if (k == 7) tmem_st_16x128b_x8(tS, &w[0]);
    if (k == 12) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        ma[e][0] = fmaxf(ma[e][0], ma[e][1]);
        ma[e][0] = fmaxf(ma[e][0], __shfl_xor_sync(0xffffffffu, ma[e][0], 1));
      }
    }
    if (k == 14) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        ma[e][0] = fmaxf(ma[e][0], __shfl_xor_sync(0xffffffffu, ma[e][0], 2));
        mxs_next[e] = ma[e][0] * c;
      }
    }
  }
  tmem_st_16x128b_x8(tS + 32, &w[16]);
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    float a0, a1;
    unpack2(add2(lacc[e][0], lacc[e][1]), a0, a1);
    l[e] += a0 + a1;
  }
}

// Output staging for a tiled store: a box of 128 rows x 32 fp32 (128-byte rows, 16-byte chunks XOR-swizzled by
// the row as the 128-byte swizzle of the tensor map expects; conflict-free for one thread per row).
__device__ __forceinline__ void stage_box_row(float* box, int r, const float (&v)[32]) {
#pragma unroll
  for (int cc = 0; cc < 8; ++cc)
    *reinterpret_cast<float4*>(box + r * 32 + ((cc ^ (r & 7)) << 2)) =
        make_float4(v[4 * cc], v[4 * cc + 1], v[4 * cc + 2], v[4 * cc + 3]);
}

}  // namespace jup
