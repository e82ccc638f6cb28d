"""jupiter_branch_append_attn_layers: one decoding / verification step for several decoder layers in one call, against
n_layers independent oracle calls (oracle.kv_append + oracle.branch per layer), and bit for bit against n_layers
single-layer calls of jupiter_branch_append_attn."""
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


def make_layers(seed, L, B, Hq, Hkv, D, P, n, lens):
    scap = int(max(lens)) + 2
    layers = []
    for l in range(L):
        s = seed + 17 * l
        q = synth.normal_bf16(s, 1, (B, n, Hq, D))
        kn, vn = synth.normal_bf16(s, 2, (B, n, Hkv, D)), synth.normal_bf16(s, 3, (B, n, Hkv, D))
        pk, pv = synth.normal_bf16(s, 4, (1, Hkv, P + 1, D)).copy(), synth.normal_bf16(s, 5, (1, Hkv, P + 1, D)).copy()
        sk, sv = synth.normal_bf16(s, 6, (B, Hkv, scap, D)).copy(), synth.normal_bf16(s, 7, (B, Hkv, scap, D)).copy()
        pk[:, :, P:], pv[:, :, P:] = 0x7FC0, 0x7F80
        for b, Lb in enumerate(lens):  # the block's rows and everything above are dead before the call
            sk[b, :, Lb - n:], sv[b, :, Lb - n:] = 0x7FC0, 0xFF80
        layers.append(dict(q=q, kn=kn, vn=vn, pk=pk, pv=pv, sk=sk, sv=sv))
    return layers, scap


def run_layers(ctx, layers, scap, B, Hq, D, P, n, lens, scale, batched):
    import torch
    import paper_2504_08242_b200 as J
    dl = torch.from_numpy(np.asarray(lens, np.int32)).cuda()
    dev, call = [], []
    for Lr in layers:
        t = {k: to_dev(v) for k, v in Lr.items()}
        t["out"] = torch.full((B, n, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
        t["lse"] = torch.full((B, Hq, n), float("nan"), dtype=torch.float32, device="cuda")
        t["pd"], t["sd"] = J.cache_desc(t["pk"], t["pv"]), J.cache_desc(t["sk"], t["sv"])
        dev.append(t)
        call.append((t["q"], t["kn"], t["vn"], t["pd"], t["sd"], t["out"], t["lse"]))
    n0 = ctx.launch_count()
    if batched:
        ctx.branch_append_attn_layers(call, P, dl, scap, B, Hq, n, scale)
    else:
        for t in dev:
            ctx.branch_append_attn(t["q"], t["kn"], t["vn"], t["pd"], P, t["sd"], dl, scap, B, Hq, n, scale, t["out"], t["lse"])
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    launches = ctx.launch_count() - n0
    return [(t["out"].cpu().numpy(), t["lse"].cpu().numpy(), to_bits(t["sk"]), to_bits(t["sv"])) for t in dev], launches


@pytest.mark.parametrize("L,B,Hq,Hkv,D,P,n,lens,one_launch", [
    (3, 8, 8, 8, 128, 300, 1, [1, 17, 64, 100, 128, 129, 200, 257], True),     # decode: streaming kernel
    (5, 4, 8, 2, 64, 77, 2, [2, 40, 90, 16], True),                            # head_dim 64, grouped heads
    (18, 2, 4, 4, 128, 40, 1, [1, 33], False),                                  # more layers than one launch holds: 2 launches
    (2, 16, 32, 8, 128, 500, 5, [5 + 21 * i for i in range(16)], False),        # verification shape: tensor-core kernel per layer
])
def test_layers_match_the_oracle_and_the_single_calls(ctx, L, B, Hq, Hkv, D, P, n, lens, one_launch):
    layers, scap = make_layers(700 + L, L, B, Hq, Hkv, D, P, n, lens)
    scale = 1.0 / np.sqrt(D)
    got, launches = run_layers(ctx, layers, scap, B, Hq, D, P, n, lens, scale, batched=True)
    one_by_one, launches1 = run_layers(ctx, layers, scap, B, Hq, D, P, n, lens, scale, batched=False)
    assert launches1 == L
    assert launches == (1 if one_launch else (2 if L == 18 else L))
    lens_np = np.asarray(lens, np.int32)
    for Lr, (out, lse, sk, sv), (out1, lse1, sk1, sv1) in zip(layers, got, one_by_one):
        rk, rv = Lr["sk"].copy(), Lr["sv"].copy()
        oracle.kv_append(rk, rv, Lr["kn"], Lr["vn"], pos_per_seq=(lens_np - n).astype(np.int32))
        ref, ref_lse = oracle.branch(Lr["q"], Lr["pk"], Lr["pv"], P, rk, rv, lens_np, scale,
                                     n_threads=oracle.hardware_threads(), return_lse=True)
        assert_close(out, ref, "layers")
        assert np.max(np.abs(lse - ref_lse)) < 2e-2
        assert np.array_equal(sk, rk) and np.array_equal(sv, rv)
        assert np.array_equal(out, out1) and np.array_equal(lse, lse1)  # same arithmetic as the single-layer call
        assert np.array_equal(sk, sk1) and np.array_equal(sv, sv1)


def test_layers_argument_errors(ctx):
    import torch
    import paper_2504_08242_b200 as J
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    B, Hq, Hkv, D, n = 2, 4, 2, 128, 1
    dl = torch.tensor([1, 5], dtype=torch.int32, device="cuda")

    def layer(cap=16, heads=Hkv):
        return (z(B, n, Hq, D), z(B, n, heads, D), z(B, n, heads, D), J.cache_desc(z(1, heads, 8, D), z(1, heads, 8, D)),
                J.cache_desc(z(B, heads, cap, D), z(B, heads, cap, D)), torch.full((B, n, Hq, D), 7.0, device="cuda"), None)
    good = [layer(), layer()]
    keep = list(good)  # (descriptors borrow the tensors)
    for layers, kw, status in [
        ([], {}, J.ERR_INVALID_ARG),
        ([layer(), layer(cap=24)], {}, J.ERR_INVALID_ARG),           # geometry differs from layer 0
        (good, dict(max_suffix_len=17), J.ERR_OUT_OF_RANGE),
        (good, dict(prefix_len=9), J.ERR_OUT_OF_RANGE),
        (good, dict(scale=float("inf")), J.ERR_INVALID_ARG),
        (good, dict(q_len=17), J.ERR_UNSUPPORTED),
    ]:
        a = dict(prefix_len=8, d_suffix_len=dl, max_suffix_len=16, n_branches=B, q_heads=Hq, q_len=n, scale=0.1)
        a.update(kw)
        n0 = ctx.launch_count()
        with pytest.raises(J.JupiterError) as e:
            ctx.branch_append_attn_layers(layers, **a)
        assert e.value.status == status and ctx.launch_count() == n0
    torch.cuda.synchronize()
    assert all(bool((l[5] == 7.0).all()) for l in keep)
