"""jupiter_chunk_prefill_append_attn (KVCache write and attention of a chunk in one call) against the
fp64 oracle: the outputs against oracle.full_causal over the whole prompt, the cache bit-exactly
against the prompt's K/V with the dead rows untouched.  Shapes are chosen to reach every launch
variant of the tensor-core kernel and the two-kernel form used for head_dim 64."""
import numpy as np
import pytest

import oracle
from workloads import synth
from tests.helpers import assert_close, run_gpu_prefill, token_to_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2504_08242_b200 as J
    c = J.Context(0)
    yield c
    c.close()


def check(ctx, w, parts, launches_per_chunk=None):
    q, k, v = w.make()
    n0 = ctx.launch_count()
    out, kc, vc, lse = run_gpu_prefill(ctx, q, k, v, parts, w.capacity, w.scale, poison=True, want_lse=True, fused=True)
    if launches_per_chunk is not None:
        assert ctx.launch_count() - n0 == launches_per_chunk * len(parts)
    ref, ref_lse = oracle.full_causal(q, k, v, w.scale, n_threads=oracle.hardware_threads(), return_lse=True)
    assert_close(out, ref, w.name)
    assert np.max(np.abs(lse - ref_lse)) < 2e-2
    S = w.seq_len
    assert np.array_equal(kc[:, :, :S], token_to_cache(k, S)) and np.array_equal(vc[:, :, :S], token_to_cache(v, S))
    assert (kc[:, :, S:] == 0x7FC0).all() and (vc[:, :, S:] == 0x7F80).all()


def test_cfg1_head_dim_64_two_kernels(ctx):
    w = synth.cfg1()
    check(ctx, w, [n for _, n in w.chunks()], launches_per_chunk=2)


def test_cfg2_one_launch_per_chunk(ctx):
    w = synth.cfg2()
    check(ctx, w, [n for _, n in w.chunks()], launches_per_chunk=1)


@pytest.mark.parametrize("parts", [[300], [1] * 5 + [295], [64, 64, 64, 64, 44], [17, 130, 3, 150], [255, 45],
                                   [129, 171]])
def test_ragged_chunkings(ctx, parts):
    S = sum(parts)
    w = synth.PrefillWorkload("fused_ragged", 160, 2, 4, 2, 128, S, S, S + 13)
    check(ctx, w, parts, launches_per_chunk=1)


def test_every_launch_variant(ctx):
    # two query tiles per CTA (grid fills the GPU), GQA, ragged
    w = synth.PrefillWorkload("fused_two_tiles", 161, 2, 32, 8, 128, 800, 800, 832)
    check(ctx, w, [100, 700], launches_per_chunk=1)
    # one query tile per CTA over several waves
    w = synth.PrefillWorkload("fused_one_tile", 162, 1, 32, 8, 128, 700, 700, 700)
    check(ctx, w, [60, 640], launches_per_chunk=1)
    # one query tile per CTA on a small grid (the loader stores the CTA's own K/V tile from its slots)
    w = synth.PrefillWorkload("fused_split", 163, 1, 8, 2, 128, 433, 433, 450)
    check(ctx, w, [64, 269, 100], launches_per_chunk=1)
    # clusters of four CTAs on a long walk: only the first CTA of a cluster writes the cache
    w = synth.PrefillWorkload("fused_cluster", 164, 1, 8, 2, 128, 3350, 3350, 3400)
    check(ctx, w, [3150, 200], launches_per_chunk=1)
    w = synth.PrefillWorkload("fused_cluster_b", 165, 1, 4, 4, 128, 3364, 3364, 3364)
    check(ctx, w, [2980, 384], launches_per_chunk=1)


def test_random_geometry(ctx):
    """Seeded random prompts: batch, head counts and group sizes, prompt lengths and ragged chunkings, so that the three
    tcgen05 forms (two query tiles per CTA, clusters, one query tile per CTA) and their boundaries are all met; both
    the fused and the two-call form, every output, LSE and the cache compared."""
    dims = synth.uniform_ints(91, 1, 10 * 6, 0, 1 << 20).reshape(-1, 6)
    for k, row in enumerate(dims):
        B = 1 + int(row[0]) % 3
        Hkv = [1, 2, 8][int(row[1]) % 3]
        G = [1, 2, 4][int(row[2]) % 3]
        S = 150 + int(row[3]) % 1300
        cuts = sorted(set(int(x) % S for x in synth.uniform_ints(int(row[4]), 2, 1 + int(row[5]) % 4, 1, 1 << 20)) - {0})
        parts = [b - a for a, b in zip([0] + cuts, cuts + [S])]
        w = synth.PrefillWorkload(f"fused_random_{k}", 700 + k, B, Hkv * G, Hkv, 128, S, S, S + int(row[5]) % 17)
        check(ctx, w, parts, launches_per_chunk=1)
        q, kk, v = w.make()
        out = run_gpu_prefill(ctx, q, kk, v, parts, w.capacity, w.scale, poison=True, fused=False)[0]
        ref = oracle.full_causal(q, kk, v, w.scale, n_threads=oracle.hardware_threads())
        assert_close(out, ref, w.name + " (two calls)")


def test_strided_cache(ctx):
    """Row stride larger than the head dimension (a cache that interleaves K and V storage)."""
    import torch
    import paper_2504_08242_b200 as J
    from tests.helpers import to_dev, to_bits
    w = synth.PrefillWorkload("fused_strided", 166, 2, 4, 2, 128, 200, 200, 208)
    q, k, v = w.make()
    B, S, Hq, D, Hkv, cap = 2, 200, 4, 128, 2, 208
    both = torch.zeros(B, Hkv, cap, 2, D, dtype=torch.bfloat16, device="cuda")
    kc, vc = both[:, :, :, 0], both[:, :, :, 1]
    desc = J.cache_desc(kc, vc)
    out = torch.full((B, S, Hq, D), float("nan"), device="cuda", dtype=torch.float32)
    pos = 0
    for n in (130, 70):
        o = torch.full((B, n, Hq, D), float("nan"), device="cuda", dtype=torch.float32)
        ctx.chunk_prefill_append_attn(to_dev(q[:, pos:pos + n]), to_dev(k[:, pos:pos + n]), to_dev(v[:, pos:pos + n]),
                                      desc, Hq, n, pos, w.scale, o)
        out[:, pos:pos + n] = o
        pos += n
    torch.cuda.synchronize()
    assert ctx.poll_device_status() == 0
    ref = oracle.full_causal(q, k, v, w.scale, n_threads=oracle.hardware_threads())
    assert_close(out.cpu().numpy(), ref, "strided")
    assert np.array_equal(to_bits(kc.contiguous())[:, :, :S], token_to_cache(k, S))
    assert np.array_equal(to_bits(vc.contiguous())[:, :, :S], token_to_cache(v, S))
    assert (to_bits(kc.contiguous())[:, :, S:] == 0).all()


def test_argument_errors(ctx):
    import torch
    import paper_2504_08242_b200 as J
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    cd = J.cache_desc(z(2, 2, 40, 128), z(2, 2, 40, 128))
    q, kn, vn = z(2, 8, 4, 128), z(2, 8, 2, 128), z(2, 8, 2, 128)
    out = torch.zeros(2, 8, 4, 128, device="cuda")
    for args, code in [((q, kn, vn, cd, 4, 8, 33, 0.1, out), J.ERR_OUT_OF_RANGE),
                       ((q, kn, vn, cd, 3, 8, 0, 0.1, out), J.ERR_INVALID_ARG),
                       ((q, None, vn, cd, 4, 8, 0, 0.1, out), J.ERR_INVALID_ARG),
                       ((q, kn, vn, cd, 4, 0, 0, 0.1, out), J.ERR_INVALID_ARG),
                       ((q, kn, vn, cd, 4, 8, 0, float("nan"), out), J.ERR_INVALID_ARG)]:
        with pytest.raises(J.JupiterError) as ei:
            ctx.chunk_prefill_append_attn(*args)
        assert ei.value.status == code
