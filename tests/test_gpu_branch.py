"""jupiter_branch_attn (+ jupiter_kv_append with per-branch positions) against the oracle."""
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
    yield c
    c.close()


def poison_dead_rows(pk, pv, P, sk, sv, lens):
    pk, pv, sk, sv = pk.copy(), pv.copy(), sk.copy(), sv.copy()
    pk[:, :, P:] = 0x7FC0
    pv[:, :, P:] = 0x7F80
    for b, L in enumerate(lens):
        sk[b, :, L:] = 0x7FC0
        sv[b, :, L:] = 0xFF80
    return pk, pv, sk, sv


def gpu_branch(ctx, q, pk, pv, P, sk, sv, lens, scale, max_len=None, want_lse=False):
    import torch
    import paper_2504_08242_b200 as J
    B, n, Hq, D = q.shape
    pkd, pvd, skd, svd = to_dev(pk), to_dev(pv), to_dev(sk), to_dev(sv)
    out = torch.full((B, n, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    lse = torch.full((B, Hq, n), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    dl = torch.from_numpy(np.asarray(lens, np.int32)).cuda()
    ctx.branch_attn(to_dev(q), J.cache_desc(pkd, pvd), P, J.cache_desc(skd, svd), dl,
                    max_len if max_len is not None else sk.shape[2], B, Hq, n, scale, out, lse)
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    return (out.cpu().numpy(), lse.cpu().numpy()) if want_lse else out.cpu().numpy()


def make_case(seed, B, Hq, Hkv, D, P, pcap, scap, n):
    q = synth.normal_bf16(seed, 1, (B, n, Hq, D))
    pk, pv = synth.normal_bf16(seed, 4, (1, Hkv, pcap, D)), synth.normal_bf16(seed, 5, (1, Hkv, pcap, D))
    sk, sv = synth.normal_bf16(seed, 6, (B, Hkv, scap, D)), synth.normal_bf16(seed, 7, (B, Hkv, scap, D))
    return q, pk, pv, sk, sv


@pytest.mark.parametrize("B,Hq,Hkv,D,P,n,lens", [
    (3, 4, 4, 64, 100, 1, [1, 40, 300]),
    (2, 8, 2, 128, 257, 5, [5, 70]),
    (5, 4, 1, 128, 64, 3, [3, 4, 256, 257, 513]),       # suffix lengths around split boundaries
    (1, 2, 2, 64, 1, 16, [16]),                          # maximal draft block, one-row prefix
    (4, 16, 2, 128, 700, 16, [16, 17, 100, 31]),         # 128 stacked rows per branch: two row tiles
    (9, 2, 2, 128, 130, 2, [2, 9, 64, 65, 66, 127, 128, 129, 200]),
])
def test_branch_small(ctx, B, Hq, Hkv, D, P, n, lens):
    scap = max(lens) + 3
    q, pk, pv, sk, sv = make_case(50 + B, B, Hq, Hkv, D, P, P + 5, scap, n)
    pk, pv, sk, sv = poison_dead_rows(pk, pv, P, sk, sv, lens)
    scale = 1.0 / np.sqrt(D)
    got, lse = gpu_branch(ctx, q, pk, pv, P, sk, sv, lens, scale, want_lse=True)
    ref, ref_lse = oracle.branch(q, pk, pv, P, sk, sv, lens, scale, return_lse=True)
    assert_close(got, ref, "branch_small")
    assert np.max(np.abs(lse - ref_lse)) < 2e-2


def test_branch_random_shapes(ctx):
    """Seeded random geometry: head counts, draft lengths, prefix and suffix lengths around tile edges."""
    shapes = synth.uniform_ints(77, 1, 6 * 8, 0, 1 << 20).reshape(-1, 8)
    for row in shapes:
        B = 1 + int(row[0]) % 9
        Hkv = [1, 2, 4][int(row[1]) % 3]
        G = [1, 2, 4, 8][int(row[2]) % 4]
        D = [64, 128][int(row[3]) % 2]
        n = 1 + int(row[4]) % 16
        P = int(row[5]) % 700
        lens = [n + int(x) % 400 for x in synth.uniform_ints(int(row[6]), 2, B, 0, 1 << 20)]
        q, pk, pv, sk, sv = make_case(100 + B, B, Hkv * G, Hkv, D, P, P + 1, max(lens) + 1, n)
        pk, pv, sk, sv = poison_dead_rows(pk, pv, P, sk, sv, lens)
        scale = 1.0 / np.sqrt(D)
        got = gpu_branch(ctx, q, pk, pv, P, sk, sv, lens, scale)
        assert_close(got, oracle.branch(q, pk, pv, P, sk, sv, lens, scale), f"random {B,Hkv,G,D,n,P,lens}")


def test_branch_without_prefix(ctx):
    B, Hq, Hkv, D, n = 3, 4, 2, 128, 4
    lens = [4, 90, 300]
    q, pk, pv, sk, sv = make_case(61, B, Hq, Hkv, D, 0, 8, 300, n)
    got = gpu_branch(ctx, q, pk, pv, 0, sk, sv, lens, 0.1)
    assert_close(got, oracle.branch(q, pk, pv, 0, sk, sv, lens, 0.1), "no_prefix")


def test_device_lengths_are_clamped(ctx):
    """A device length outside [q_len, max_suffix_len] is clamped before use."""
    B, Hq, Hkv, D, P, n = 2, 2, 2, 64, 50, 2
    q, pk, pv, sk, sv = make_case(62, B, Hq, Hkv, D, P, P, 40, n)
    got = gpu_branch(ctx, q, pk, pv, P, sk, sv, [0, 1000], 0.125, max_len=40)
    ref = oracle.branch(q, pk, pv, P, sk, sv, [2, 40], 0.125)
    assert_close(got, ref, "clamped")


def test_cfg4_outline_decode_steps(ctx):
    """Shared 1024-row prefix, 8 branches, 1 query per branch; 64 steps each appending one
    K/V row per branch at its own position, then attending.  Every step is checked."""
    import torch
    import paper_2504_08242_b200 as J
    w = synth.cfg4()
    pk, pv, sk, sv = w.make_caches()
    hist = w.history_lengths()
    pk_d, pv_d, sk_d, sv_d = to_dev(pk), to_dev(pv), to_dev(sk), to_dev(sv)
    pdesc, sdesc = J.cache_desc(pk_d, pv_d), J.cache_desc(sk_d, sv_d)
    out = torch.empty(w.n_branches, 1, w.q_heads, w.head_dim, dtype=torch.float32, device="cuda")
    sk_ref, sv_ref = sk.copy(), sv.copy()
    worst = (0.0, 0.0)
    for t in range(w.steps):
        q, kn, vn = w.make_step(t)
        pos = (hist + t).astype(np.int32)
        lens = pos + 1
        ctx.kv_append(sdesc, to_dev(kn), to_dev(vn), 1, 0, torch.from_numpy(pos).cuda())
        ctx.branch_attn(to_dev(q), pdesc, w.prefix_len, sdesc, torch.from_numpy(lens).cuda(),
                        w.suffix_capacity, w.n_branches, w.q_heads, 1, w.scale, out)
        oracle.kv_append(sk_ref, sv_ref, kn, vn, pos_per_seq=pos)
        ref = oracle.branch(q, pk, pv, w.prefix_len, sk_ref, sv_ref, lens, w.scale,
                            n_threads=oracle.hardware_threads())
        mx, fro = assert_close(out.cpu().numpy(), ref, f"cfg4 step {t}")
        worst = (max(worst[0], mx), max(worst[1], fro))
    assert np.array_equal(to_bits(sk_d), sk_ref) and np.array_equal(to_bits(sv_d), sv_ref)


def test_cfg5_speculative_verification(ctx):
    import torch
    import paper_2504_08242_b200 as J
    w = synth.cfg5()
    pk, pv, sk, sv = w.make_caches()
    hist = w.history_lengths()
    q, kn, vn = w.make_step(0)
    lens = (hist + w.q_len).astype(np.int32)
    pk, pv, sk, sv = poison_dead_rows(pk, pv, w.prefix_len, sk, sv, lens)
    pk_d, pv_d, sk_d, sv_d = to_dev(pk), to_dev(pv), to_dev(sk), to_dev(sv)
    sdesc = J.cache_desc(sk_d, sv_d)
    out = torch.empty(w.n_branches, w.q_len, w.q_heads, w.head_dim, dtype=torch.float32, device="cuda")
    ctx.kv_append(sdesc, to_dev(kn), to_dev(vn), w.q_len, 0, torch.from_numpy(hist.astype(np.int32)).cuda())
    ctx.branch_attn(to_dev(q), J.cache_desc(pk_d, pv_d), w.prefix_len, sdesc, torch.from_numpy(lens).cuda(),
                    int(lens.max()), w.n_branches, w.q_heads, w.q_len, w.scale, out)
    torch.cuda.synchronize()
    oracle.kv_append(sk, sv, kn, vn, pos_per_seq=hist)
    ref = oracle.branch(q, pk, pv, w.prefix_len, sk, sv, lens, w.scale, n_threads=oracle.hardware_threads())
    assert_close(out.cpu().numpy(), ref, "cfg5")


def test_branch_repeatable(ctx):
    B, Hq, Hkv, D, P, n = 4, 8, 2, 128, 600, 5
    lens = [5, 300, 17, 280]
    q, pk, pv, sk, sv = make_case(63, B, Hq, Hkv, D, P, P, 300, n)
    a = gpu_branch(ctx, q, pk, pv, P, sk, sv, lens, 0.09)
    b = gpu_branch(ctx, q, pk, pv, P, sk, sv, lens, 0.09)
    assert np.array_equal(a, b)


def test_branch_argument_errors(ctx):
    import torch
    import paper_2504_08242_b200 as J
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    pd = J.cache_desc(z(1, 2, 32, 64), z(1, 2, 32, 64))
    sd = J.cache_desc(z(3, 2, 20, 64), z(3, 2, 20, 64))
    q = z(3, 2, 4, 64)
    out = torch.full((3, 2, 4, 64), 7.0, dtype=torch.float32, device="cuda")
    dl = torch.full((3,), 2, dtype=torch.int32, device="cuda")
    cases = [
        (dict(prefix_len=33), J.ERR_OUT_OF_RANGE),
        (dict(max_suffix_len=21), J.ERR_OUT_OF_RANGE),
        (dict(max_suffix_len=1), J.ERR_OUT_OF_RANGE),
        (dict(n_branches=2), J.ERR_INVALID_ARG),
        (dict(q_len=17, max_suffix_len=20), J.ERR_UNSUPPORTED),
        (dict(q_heads=3), J.ERR_INVALID_ARG),
        (dict(d_suffix_len=None), J.ERR_INVALID_ARG),
    ]
    for over, status in cases:
        a = dict(q=q, prefix=pd, prefix_len=32, suffix=sd, d_suffix_len=dl, max_suffix_len=20, n_branches=3,
                 q_heads=4, q_len=2, scale=0.125, out=out)
        a.update(over)
        with pytest.raises(J.JupiterError) as e:
            ctx.branch_attn(**a)
        assert e.value.status == status, over
    # only the split-KV kernel keeps partial results in the context's scratch: a context with too little of it
    # refuses that kernel and still serves the shapes that the streaming kernel takes
    small = J.Context(0, workspace_bytes=1024)
    small.select_branch_kernel(J.BRANCH_SPLIT_KV)
    with pytest.raises(J.JupiterError) as e:
        small.branch_attn(q, pd, 32, sd, dl, 20, 3, 4, 2, 0.125, out)
    assert e.value.status == J.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    small.select_branch_kernel(J.BRANCH_AUTO)
    small.branch_attn(q, pd, 32, sd, dl, 20, 3, 4, 2, 0.125, out)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(out).all()) and not bool((out == 7.0).all())
    out.fill_(7.0)
    small.close()
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
