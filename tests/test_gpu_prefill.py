"""jupiter_chunk_prefill_attn (+ jupiter_kv_append) against the fp64 oracle.

Small and ragged shapes are compared element by element; the 8192-token workload is
compared on sampled rows the oracle computes one by one.  Tolerance: max-abs <= 1e-2 and
relative Frobenius <= 5e-3 (bf16 inputs, fp32 accumulation)."""
import numpy as np
import pytest

import oracle
from workloads import synth
from tests.helpers import assert_close, run_gpu_prefill, to_dev, token_to_cache

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2504_08242_b200 as J
    c = J.Context(0)
    yield c
    c.close()


def check_workload(ctx, w, parts=None, want_lse=False):
    q, k, v = w.make()
    parts = parts or [n for _, n in w.chunks()]
    res = run_gpu_prefill(ctx, q, k, v, parts, w.capacity, w.scale, poison=True, want_lse=want_lse)
    ref, ref_lse = oracle.full_causal(q, k, v, w.scale, n_threads=oracle.hardware_threads(), return_lse=True)
    assert_close(res[0], ref, w.name)
    # the cache ends up holding exactly the prompt's K/V (bit-exact), dead rows untouched
    S = w.seq_len
    assert np.array_equal(res[1][:, :, :S], token_to_cache(k, S)) and np.array_equal(res[2][:, :, :S], token_to_cache(v, S))
    assert (res[1][:, :, S:] == 0x7FC0).all() and (res[2][:, :, S:] == 0x7F80).all()
    if want_lse:
        assert np.max(np.abs(res[3] - ref_lse)) < 2e-2
    return res


def test_cfg1_tiny_prefill(ctx):
    check_workload(ctx, synth.cfg1(), want_lse=True)


def test_cfg2_7b_shaped_prefill(ctx):
    check_workload(ctx, synth.cfg2())


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("parts", [[300], [1] * 9 + [291], [64, 64, 64, 64, 44], [17, 130, 3, 150], [255, 45],
                                   [129, 171]])
def test_ragged_chunkings(ctx, D, parts):
    S = sum(parts)
    w = synth.PrefillWorkload(f"ragged_D{D}", 30 + D, 2, 4, 2, D, S, S, S + 13)
    check_workload(ctx, w, parts=parts, want_lse=True)


def test_pure_decode_steps_after_a_chunk(ctx):
    # chunk size 1 is token-by-token decoding against the growing cache
    w = synth.PrefillWorkload("decode_tail", 41, 1, 8, 8, 128, 96, 96, 96)
    check_workload(ctx, w, parts=[70] + [1] * 26)


def test_gqa_group_of_eight(ctx):
    w = synth.PrefillWorkload("gqa8", 42, 1, 16, 2, 128, 200, 200, 256)
    check_workload(ctx, w, parts=[128, 72])


def test_two_query_tiles_per_cta_ragged(ctx):
    """Enough (sequence, head, 256-row block) units to fill the GPU, so the kernel variant with two
    query tiles per CTA runs; ragged chunk lengths and positions, every output compared."""
    w = synth.PrefillWorkload("two_tiles", 45, 2, 32, 8, 128, 800, 800, 832)
    check_workload(ctx, w, parts=[100, 700], want_lse=True)
    w = synth.PrefillWorkload("two_tiles_b", 46, 3, 32, 32, 128, 515, 515, 515)
    check_workload(ctx, w, parts=[515])


def test_one_query_tile_per_cta_small_grids(ctx):
    """Few (sequence, head, 128-row tile) units: one query tile per CTA, both softmax warpgroups on it (16 rows per
    warp).  Covers walks of one, two and three tiles (the pipeline holds three score buffers; the last three tiles
    complete the accumulator's own barriers), rows that see none of the last tile (position not a multiple of
    128), a ragged last query tile, GQA, and LSE."""
    w = synth.PrefillWorkload("frag_a", 48, 1, 8, 2, 128, 433, 433, 450)
    check_workload(ctx, w, parts=[64, 269, 100], want_lse=True)
    w = synth.PrefillWorkload("frag_b", 49, 2, 4, 4, 128, 1100, 1100, 1100)
    check_workload(ctx, w, parts=[1, 127, 130, 842], want_lse=True)


@pytest.mark.parametrize("tiles", [1, 2, 3, 4, 5, 7])
def test_one_query_tile_per_cta_walk_lengths(ctx, tiles):
    """Every short walk length of the three-buffer pipeline, one call on a cold cache (the unfused call must leave the
    cache untouched: check_workload compares it bit by bit afterwards)."""
    S = tiles * 128 - 37
    w = synth.PrefillWorkload(f"frag_walk_{tiles}", 170 + tiles, 1, 2, 1, 128, S, S, S + 5)
    first = max(S - 100, 1)
    check_workload(ctx, w, parts=[first, S - first] if S > first else [S], want_lse=True)


def test_one_query_tile_per_cta_more_tiles_than_sms(ctx):
    """More 128-row tiles than SMs but too few 256-row pairs to fill them: the same form over several waves."""
    w = synth.PrefillWorkload("one_tile", 50, 1, 32, 8, 128, 700, 700, 700)
    check_workload(ctx, w, parts=[60, 640])


def test_cluster_shares_a_long_walk(ctx):
    """A long KV walk on a small grid: clusters of four CTAs take every fourth KV tile and exchange
    partial (O, m, l).  Ragged position and chunk length (the last tiles are hidden from early rows, one
    CTA of a cluster can be left without visible keys for a row), a block whose second query tile does
    not exist (384 rows), GQA, and LSE."""
    w = synth.PrefillWorkload("cluster_a", 51, 1, 8, 2, 128, 3350, 3350, 3400)
    check_workload(ctx, w, parts=[3150, 200], want_lse=True)
    w = synth.PrefillWorkload("cluster_b", 52, 1, 4, 4, 128, 3364, 3364, 3364)
    check_workload(ctx, w, parts=[2980, 384], want_lse=True)
    w = synth.PrefillWorkload("cluster_c", 53, 2, 8, 8, 128, 3328, 3328, 3328)
    check_workload(ctx, w, parts=[3072, 256], want_lse=True)


def test_negative_scale_uses_the_general_kernel(ctx):
    """scale <= 0 is legal (softmax of the negated scores); head_dim 128 then takes the mma.sync path."""
    import torch
    import paper_2504_08242_b200 as J
    w = synth.PrefillWorkload("neg_scale", 47, 1, 4, 2, 128, 200, 200, 200)
    q, k, v = w.make()
    res = run_gpu_prefill(ctx, q, k, v, [77, 123], 200, -0.05, poison=True)
    assert_close(res[0], oracle.full_causal(q, k, v, -0.05), "negative scale")


def test_strided_cache_rows(ctx):
    """stride_row > D and a cache that is a view into a larger allocation."""
    import torch
    import paper_2504_08242_b200 as J
    B, S, H, D, cap = 1, 130, 2, 64, 140
    w = synth.PrefillWorkload("strided", 43, B, H, H, D, S, S, cap)
    q, k, v = w.make()
    big_k = torch.full((B, H, cap, D + 8), float("nan"), dtype=torch.bfloat16, device="cuda")
    big_v = torch.full((B, H, cap, D + 8), float("nan"), dtype=torch.bfloat16, device="cuda")
    desc = J.cache_desc(big_k[..., :D], big_v[..., :D])
    ctx.kv_append(desc, to_dev(k), to_dev(v), S, 0)
    out = torch.empty(B, S, H, D, dtype=torch.float32, device="cuda")
    ctx.chunk_prefill_attn(to_dev(q), desc, H, S, 0, w.scale, out)
    torch.cuda.synchronize()
    assert_close(out.cpu().numpy(), oracle.full_causal(q, k, v, w.scale), "strided")


def test_results_are_run_to_run_identical(ctx):
    w = synth.PrefillWorkload("repeat", 44, 1, 4, 4, 128, 256, 128, 256)
    q, k, v = w.make()
    a = run_gpu_prefill(ctx, q, k, v, [128, 128], 256, w.scale)[0]
    b = run_gpu_prefill(ctx, q, k, v, [128, 128], 256, w.scale)[0]
    assert np.array_equal(a, b)


def _cfg3_sampled_rows(w, q, k, v, out, chunk):
    """The oracle evaluates sampled (sequence, head, row) outputs of the full-size workload one by one."""
    G = w.q_heads // w.kv_heads
    rows = [(0, 0, 0), (3, 31, 8191), (1, 5, chunk - 1), (2, 17, chunk), (0, 9, 4095), (3, 2, 8191 - chunk)]
    pick = synth.uniform_ints(99, 1, 3 * 58, 0, 1 << 30).reshape(-1, 3)
    rows += [(int(a) % w.batch, int(b) % w.q_heads, int(c) % w.seq_len) for a, b, c in pick]
    got, ref = [], []
    for b, h, i in rows:
        kk = np.ascontiguousarray(k[b, :i + 1, h // G])
        vv = np.ascontiguousarray(v[b, :i + 1, h // G])
        o, _ = oracle.attend(q[b, i, h], kk, vv, w.scale)
        ref.append(o)
        got.append(out[b, i, h])
    assert_close(np.array(got), np.array(ref), w.name)


@pytest.mark.parametrize("chunk", [128, 512, 1024])
def test_cfg3_gqa_long_prompt_sampled_rows(ctx, chunk):
    """Full 4 x 8192-token GQA prompt on the GPU through the two-call form (jupiter_kv_append, then
    jupiter_chunk_prefill_attn per chunk)."""
    w = synth.cfg3(chunk)
    q, k, v = w.make()
    out = run_gpu_prefill(ctx, q, k, v, [n for _, n in w.chunks()], w.capacity, w.scale, poison=False)[0]
    assert np.isfinite(out).all()
    _cfg3_sampled_rows(w, q, k, v, out, chunk)


@pytest.mark.parametrize("chunk", [128, 512, 1024])
def test_cfg3_fused_sampled_rows(ctx, chunk):
    """The same workload in the launch configuration the benchmark times: one jupiter_chunk_prefill_append_attn call
    per chunk (batch 4, GQA, 64 / 16 / 8 launches walking up to 64 KV tiles).  Sampled outputs against the oracle,
    and the final caches bit for bit against the prompt's K/V (dead rows, poisoned beforehand, included)."""
    from tests.helpers import token_to_cache
    w = synth.cfg3(chunk)
    q, k, v = w.make()
    cap = w.capacity + 128  # rows above the prompt stay poisoned
    out, kc, vc = run_gpu_prefill(ctx, q, k, v, [n for _, n in w.chunks()], cap, w.scale, poison=True, fused=True)
    assert np.isfinite(out).all()
    _cfg3_sampled_rows(w, q, k, v, out, chunk)
    assert np.array_equal(kc, token_to_cache(k, cap, 0x7FC0)) and np.array_equal(vc, token_to_cache(v, cap, 0x7F80))


def test_prefill_argument_errors(ctx):
    import torch
    import paper_2504_08242_b200 as J
    kc = torch.zeros(1, 2, 64, 64, dtype=torch.bfloat16, device="cuda")
    d = J.cache_desc(kc, torch.zeros_like(kc))
    q = torch.zeros(1, 8, 4, 64, dtype=torch.bfloat16, device="cuda")
    out = torch.full((1, 8, 4, 64), 7.0, dtype=torch.float32, device="cuda")
    for args, status in [
        ((q, d, 4, 8, 60, 0.125, out), J.ERR_OUT_OF_RANGE),   # pos + q_len > capacity
        ((q, d, 3, 8, 0, 0.125, out), J.ERR_INVALID_ARG),     # 3 query heads over 2 KV heads
        ((q, d, 4, 0, 0, 0.125, out), J.ERR_INVALID_ARG),     # empty chunk
        ((None, d, 4, 8, 0, 0.125, out), J.ERR_INVALID_ARG),
        ((q, d, 4, 8, 0, float("nan"), out), J.ERR_INVALID_ARG),
    ]:
        with pytest.raises(J.JupiterError) as e:
            ctx.chunk_prefill_attn(*args)
        assert e.value.status == status
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
