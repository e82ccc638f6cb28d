"""The tensor-core (tcgen05 / TMEM) branch-attention kernel, pinned with jupiter_select_branch_kernel, against the
oracle: plain, fused KVCache write and token-tree calls on the geometries that steer it -- one partial row tile,
full tiles with a ragged tail, branches that straddle two row tiles, prefix and suffix lengths around the 128-key
tile edges, no prefix, one or several CTAs per (kv head, row tile) unit, dead rows holding NaN / Inf."""
import numpy as np
import pytest

import oracle
from workloads import synth
from tests.helpers import assert_close, to_dev, to_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2504_08242_b200 as J
    c = J.Context(0)
    c.select_branch_kernel(J.BRANCH_TENSOR_CORE)
    yield c
    c.close()


def random_tree_masks(seed, B, n):
    picks = synth.uniform_ints(seed, 5, B * n, 0, 1 << 20).reshape(B, n)
    tm = np.zeros((B, n), np.uint32)
    for b in range(B):
        for i in range(n):
            parent = int(picks[b, i]) % (i + 1) - 1
            tm[b, i] = (tm[b, parent] if parent >= 0 else 0) | (1 << i)
    return tm


def run_case(ctx, seed, B, Hq, Hkv, P, n, lens, mode="plain", scale=None, check_lse=True):
    """mode: plain (rows already in the cache), fused (block written by the call), tree (ancestor masks)."""
    import torch
    import paper_2504_08242_b200 as J
    D = 128
    lens = np.asarray(lens, np.int32)
    scap = int(lens.max()) + 3
    scale = 1.0 / np.sqrt(D) if scale is None else scale
    q = synth.normal_bf16(seed, 1, (B, n, Hq, D))
    kn, vn = synth.normal_bf16(seed, 2, (B, n, Hkv, D)), synth.normal_bf16(seed, 3, (B, n, Hkv, D))
    pk, pv = synth.normal_bf16(seed, 4, (1, Hkv, P + 2, D)).copy(), synth.normal_bf16(seed, 5, (1, Hkv, P + 2, D)).copy()
    sk, sv = synth.normal_bf16(seed, 6, (B, Hkv, scap, D)).copy(), synth.normal_bf16(seed, 7, (B, Hkv, scap, D)).copy()
    pk[:, :, P:], pv[:, :, P:] = 0x7FC0, 0x7F80
    for b, L in enumerate(lens):  # dead rows are poison; with the fused write the block's rows are dead before the call
        first_dead = L - n if mode == "fused" else L
        sk[b, :, first_dead:], sv[b, :, first_dead:] = 0x7FC0, 0xFF80
    rk, rv = sk.copy(), sv.copy()
    if mode == "fused":
        oracle.kv_append(rk, rv, kn, vn, pos_per_seq=(lens - n).astype(np.int32))
    tm = random_tree_masks(seed + 1, B, n) if mode == "tree" else None
    nt = oracle.hardware_threads()
    if mode == "tree":
        ref, ref_lse = oracle.branch_tree(q, pk, pv, P, rk, rv, lens, tm, scale, n_threads=nt, return_lse=True)
    else:
        ref, ref_lse = oracle.branch(q, pk, pv, P, rk, rv, lens, scale, n_threads=nt, return_lse=True)
    pkd, pvd, skd, svd = to_dev(pk), to_dev(pv), to_dev(sk), to_dev(sv)
    pd, sd = J.cache_desc(pkd, pvd), J.cache_desc(skd, svd)
    out = torch.full((B, n, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B, Hq, n), float("nan"), dtype=torch.float32, device="cuda")
    dl = torch.from_numpy(lens).cuda()
    n0 = ctx.launch_count()
    if mode == "fused":
        ctx.branch_append_attn(to_dev(q), to_dev(kn), to_dev(vn), pd, P, sd, dl, scap, B, Hq, n, scale, out, lse)
    elif mode == "tree":
        ctx.branch_attn_tree(to_dev(q), pd, P, sd, dl, torch.from_numpy(tm.view(np.int32)).cuda(), scap, B, Hq, n, scale,
                             out, lse)
    else:
        ctx.branch_attn(to_dev(q), pd, P, sd, dl, scap, B, Hq, n, scale, out, lse)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    assert ctx.launch_count() - n0 == 1
    assert_close(out.cpu().numpy(), ref, f"branch_tc {mode}")
    if check_lse:
        assert np.max(np.abs(lse.cpu().numpy() - ref_lse)) < 2e-2
    assert np.array_equal(to_bits(skd), rk) and np.array_equal(to_bits(svd), rv)  # only the block's rows were written
    return out.cpu().numpy()


SHAPES = [
    # B, Hq, Hkv, P, n, lens
    (2, 8, 2, 257, 5, [5, 70]),                                   # 40 rows: one partial row tile
    (4, 16, 2, 700, 16, [16, 17, 100, 31]),                       # 128 rows per branch: tiles = branches... 512 rows
    (7, 8, 2, 300, 5, [5, 127, 128, 129, 255, 256, 257]),         # 140 rows: a branch straddles the tile edge
    (16, 32, 8, 600, 5, [5 + 19 * i for i in range(16)]),         # the verification shape, 320 rows per kv head
    (3, 4, 4, 0, 8, [8, 200, 390]),                               # no prefix, MHA (G = 1)
    (5, 8, 1, 128, 3, [3, 4, 130, 131, 260]),                     # prefix of exactly one tile, G = 8
    (2, 2, 2, 1, 16, [16, 144]),                                  # one-row prefix, maximal draft block
    (26, 4, 4, 2048, 5, [5 + 3 * i for i in range(26)]),          # n G = 5: 26 branches inside one row tile
    (9, 128, 1, 90, 1, [1, 2, 3, 64, 128, 129, 300, 301, 77]),    # G = 128: a row tile is one token
]


@pytest.mark.parametrize("B,Hq,Hkv,P,n,lens", SHAPES)
def test_branch_tc(ctx, B, Hq, Hkv, P, n, lens):
    run_case(ctx, 400 + B + n, B, Hq, Hkv, P, n, lens, "plain")


@pytest.mark.parametrize("B,Hq,Hkv,P,n,lens", SHAPES)
def test_branch_tc_fused_write(ctx, B, Hq, Hkv, P, n, lens):
    run_case(ctx, 420 + B + n, B, Hq, Hkv, P, n, lens, "fused")


@pytest.mark.parametrize("B,Hq,Hkv,P,n,lens", SHAPES[:6])
def test_branch_tc_tree(ctx, B, Hq, Hkv, P, n, lens):
    run_case(ctx, 440 + B + n, B, Hq, Hkv, P, n, lens, "tree")


@pytest.mark.parametrize("mode", ["plain", "fused", "tree"])
def test_one_cta_per_unit(ctx, mode):
    """More (kv head, row tile) units than half the SMs: every unit is walked by a single CTA (no cluster)."""
    lens = [5 + (37 * i) % 300 for i in range(30)]
    run_case(ctx, 460, 30, 64, 16, 300, 5, lens, mode)


def test_a_branch_larger_than_a_row_tile(ctx):
    """q_len x group = 256 stacked rows per branch: two 128-row slices of one branch per kv head, the first of
    which writes the block into the cache."""
    for mode in ("plain", "fused", "tree"):
        run_case(ctx, 465, 3, 32, 2, 200, 16, [16, 150, 300], mode)


def test_group_sizes_that_are_not_powers_of_two(ctx):
    run_case(ctx, 466, 5, 6, 2, 130, 4, [4, 60, 129, 200, 7], "fused")      # group 3: 12 rows per branch
    run_case(ctx, 467, 4, 10, 2, 260, 3, [3, 128, 131, 40], "tree")         # group 5


def test_random_geometry(ctx):
    """Seeded random shapes: head counts and group sizes (powers of two or not), draft lengths, prefix and suffix lengths
    around tile edges, few or many branches; every call mode."""
    shapes = synth.uniform_ints(78, 1, 10 * 8, 0, 1 << 20).reshape(-1, 8)
    for k, row in enumerate(shapes):
        B = 1 + int(row[0]) % 20
        Hkv = [1, 2, 4][int(row[1]) % 3]
        G = [1, 2, 3, 4, 8][int(row[2]) % 5]
        n = 1 + int(row[3]) % 16
        P = [0, 1, 127, 128, 129, 500, 1100][int(row[4]) % 7]
        lens = [n + int(x) % 420 for x in synth.uniform_ints(int(row[5]), 2, B, 0, 1 << 20)]
        mode = ["plain", "fused", "tree"][k % 3]
        run_case(ctx, 600 + k, B, Hkv * G, Hkv, P, n, lens, mode)


def test_block_straddles_key_tiles(ctx):
    """The draft block crosses a 128-key tile edge: its rows are patched into two tiles."""
    for L in (129, 130, 131, 132, 256 + 2):
        run_case(ctx, 470 + L, 3, 8, 2, 64, 5, [L, L + 1, 5], "fused")
        run_case(ctx, 480 + L, 3, 8, 2, 64, 5, [L, L + 1, 5], "tree")


def test_long_walk_many_tiles(ctx):
    """Every CTA lists more tiles than its rings hold many times over (ring reuse, barrier parities)."""
    run_case(ctx, 490, 4, 8, 2, 9000, 4, [4, 2500, 4100, 129], "fused")
    lens = [5 + (41 * i) % 900 for i in range(30)]
    run_case(ctx, 491, 30, 64, 16, 1500, 5, lens, "fused")  # single-CTA units


def test_repeatable_and_matches_the_other_kernels(ctx):
    """Fixed merge order: two runs give identical bits; the split-KV kernel agrees within the tolerance."""
    import paper_2504_08242_b200 as J
    args = (500, 16, 32, 8, 900, 5, [5 + 23 * i for i in range(16)])
    a = run_case(ctx, *args, "fused")
    b = run_case(ctx, *args, "fused")
    assert np.array_equal(a, b)
    other = J.Context(0)
    other.select_branch_kernel(J.BRANCH_SPLIT_KV)
    import torch
    try:
        D = 128
        seed, B, Hq, Hkv, P, n, lens = args
        lens = np.asarray(lens, np.int32)
        scap = int(lens.max()) + 3
        q = synth.normal_bf16(seed, 1, (B, n, Hq, D))
        kn, vn = synth.normal_bf16(seed, 2, (B, n, Hkv, D)), synth.normal_bf16(seed, 3, (B, n, Hkv, D))
        pk, pv = synth.normal_bf16(seed, 4, (1, Hkv, P + 2, D)), synth.normal_bf16(seed, 5, (1, Hkv, P + 2, D))
        sk, sv = synth.normal_bf16(seed, 6, (B, Hkv, scap, D)), synth.normal_bf16(seed, 7, (B, Hkv, scap, D))
        out = torch.empty(B, n, Hq, D, dtype=torch.float32, device="cuda")
        pkd, pvd, skd, svd = to_dev(pk), to_dev(pv), to_dev(sk), to_dev(sv)  # (kept alive: a descriptor borrows)
        other.branch_append_attn(to_dev(q), to_dev(kn), to_dev(vn), J.cache_desc(pkd, pvd), P, J.cache_desc(skd, svd),
                                 torch.from_numpy(lens).cuda(), scap, B, Hq, n, 1.0 / np.sqrt(D), out)
        torch.cuda.synchronize()
        assert np.max(np.abs(out.cpu().numpy() - a)) < 1e-2
    finally:
        other.close()


def test_unsupported_shapes_are_refused_when_pinned(ctx):
    import torch
    import paper_2504_08242_b200 as J
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    dl = torch.full((2,), 4, dtype=torch.int32, device="cuda")
    for Hq, Hkv, D, n in [(4, 2, 64, 4),      # head_dim 64
                          (34, 2, 128, 16)]:  # 272 rows per branch and a group of 17, which does not divide 128
        pd = J.cache_desc(z(1, Hkv, 32, D), z(1, Hkv, 32, D))
        sd = J.cache_desc(z(2, Hkv, 40, D), z(2, Hkv, 40, D))
        out = torch.zeros(2, n, Hq, D, device="cuda")
        with pytest.raises(J.JupiterError) as e:
            ctx.branch_attn(z(2, n, Hq, D), pd, 32, sd, dl, 40, 2, Hq, n, 0.1, out)
        assert e.value.status == J.ERR_UNSUPPORTED
    with pytest.raises(J.JupiterError) as e:   # a non-positive scale takes the general kernels
        pd = J.cache_desc(z(1, 2, 32, 128), z(1, 2, 32, 128))
        sd = J.cache_desc(z(2, 2, 40, 128), z(2, 2, 40, 128))
        ctx.branch_attn(z(2, 4, 8, 128), pd, 32, sd, dl, 40, 2, 8, 4, -0.1, torch.zeros(2, 4, 8, 128, device="cuda"))
    assert e.value.status == J.ERR_UNSUPPORTED
