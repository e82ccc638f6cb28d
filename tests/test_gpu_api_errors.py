"""Argument errors common to the attention entry points: a softmax scale that is not a finite number and a cache
descriptor with a zero stride on a dimension that has more than one entry are refused on the host, before anything
is enqueued, with the outputs untouched."""
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2504_08242_b200 as J
    c = J.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("scale", [float("inf"), float("-inf"), float("nan")])
def test_non_finite_scale_is_refused_everywhere(ctx, scale):
    import torch
    import paper_2504_08242_b200 as J
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    for D in (64, 128):
        cache = J.cache_desc(z(2, 2, 64, D), z(2, 2, 64, D))
        pfx = J.cache_desc(z(1, 2, 32, D), z(1, 2, 32, D))
        q, kn, vn = z(2, 8, 4, D), z(2, 8, 2, D), z(2, 8, 2, D)
        out = torch.full((2, 8, 4, D), 7.0, device="cuda")
        dl = torch.full((2,), 8, dtype=torch.int32, device="cuda")
        tm = torch.full((2, 8), 255, dtype=torch.int32, device="cuda")
        n0 = ctx.launch_count()
        calls = [
            lambda: ctx.chunk_prefill_attn(q, cache, 4, 8, 0, scale, out),
            lambda: ctx.chunk_prefill_append_attn(q, kn, vn, cache, 4, 8, 0, scale, out),
            lambda: ctx.branch_attn(q, pfx, 32, cache, dl, 64, 2, 4, 8, scale, out),
            lambda: ctx.branch_append_attn(q, kn, vn, pfx, 32, cache, dl, 64, 2, 4, 8, scale, out),
            lambda: ctx.branch_attn_tree(q, pfx, 32, cache, dl, tm, 64, 2, 4, 8, scale, out),
            lambda: J.branch_attn_noalloc(q, pfx, 32, cache, dl, 64, 2, 4, 8, scale, out),
        ]
        if D == 128:
            calls.append(lambda: ctx.branch_prefill_attn(q, pfx, 32, cache, 4, 8, 0, scale, out))
        for call in calls:
            with pytest.raises(J.JupiterError) as e:
                call()
            assert e.value.status == J.ERR_INVALID_ARG
        assert ctx.launch_count() == n0
        torch.cuda.synchronize()
        assert bool((out == 7.0).all())


def test_broadcast_cache_is_refused(ctx):
    """stride 0 over several heads or sequences cannot be encoded in a tensor map: refused, not misread."""
    import torch
    import paper_2504_08242_b200 as J
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    k, v = z(2, 2, 64, 128), z(2, 2, 64, 128)
    q = z(2, 8, 4, 128)
    out = torch.full((2, 8, 4, 128), 7.0, device="cuda")
    for field in ("stride_batch", "stride_head"):
        d = J.cache_desc(k, v)
        setattr(d, field, 0)
        with pytest.raises(J.JupiterError) as e:
            ctx.chunk_prefill_attn(q, d, 4, 8, 0, 0.1, out)
        assert e.value.status == J.ERR_INVALID_ARG
    one = J.cache_desc(z(1, 1, 64, 128), z(1, 1, 64, 128))  # extent-1 dimensions may carry any stride
    one.stride_batch = 0
    one.stride_head = 0
    o1 = torch.zeros(1, 8, 1, 128, device="cuda")
    ctx.chunk_prefill_attn(z(1, 8, 1, 128), one, 1, 8, 0, 0.1, o1)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
