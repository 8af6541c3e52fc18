"""kvq_decode_attn_static: decode attention for callers that must not allocate.

A serving loop under a "no allocation after start-up" rule, or a plug-in living inside a
process whose device memory belongs to another allocator, cannot let a library reserve scratch
for it.  This entry point keeps the split-attention partials in a fixed array inside the library
image instead, so the call itself performs no allocation.  The test drives it through the C ABI
and checks that it returns exactly what kvq_decode_attn returns (bit for bit: the same kernel runs
with the same plan) and that both agree with the CPU oracle -- twice in a row, because the array
is shared by all calls and keeps the previous call's contents, and once more on a different cache
so that stale partials of a larger problem cannot leak into a smaller one.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest

from paper_2604_04722_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_04722_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _filled_cache(gu, oracle, batch, q_heads, kv_heads, n, seed):
    K, V = synth.kv_batch(seed, 0, batch, 0, n, kv_heads)
    bits = np.stack([synth.bits_iid(seed, b, 0, n, (0.4, 0.3, 0.2, 0.1)) for b in range(batch)])
    g = gu.GpuCache(1, batch, q_heads, kv_heads, n)
    g.append(0, K, V, bits)
    oc = None
    if oracle is not None:
        oc = oracle.OracleCache(batch, q_heads, kv_heads)
        oc.append(K, V, bits)
    return g, oc


def _both(gu, g, Q):
    import torch
    from paper_2604_04722_b200 import binding as kq
    Qd = gu.dev(Q.view(np.uint16))
    want = torch.zeros_like(Qd)
    kq.kvq_decode_attn(g.ctx, 0, Qd, want)
    outs = []
    for _ in range(2):                                   # two calls in a row share the array
        got = torch.full_like(Qd, 0x7e00)                # fp16 NaN pattern: every element must be written
        kq.kvq_decode_attn_static(g.ctx, 0, Qd, got)
        outs.append(got)
    torch.cuda.synchronize()
    return want.cpu().numpy().view(np.uint16), [o.cpu().numpy().view(np.uint16) for o in outs]


def test_static_scratch_entry_matches_the_allocating_one_twice_in_a_row(gu, oracle):
    """Same kernel, same launch plan, only the scratch differs: the two entry points must agree BIT FOR BIT
    (a tolerance would hide a stale partial or a counter left behind), and both lie within the attention
    tolerance of the oracle."""
    from paper_2604_04722_b200 import binding as kq
    big, oc_big = _filled_cache(gu, oracle, 4, 6, 2, 3000, seed=11)       # several splits, ragged last tiles
    small, oc_small = _filled_cache(gu, oracle, 2, 3, 3, 70, seed=12)     # a smaller problem afterwards
    try:
        for g, oc, step in ((big, oc_big, 0), (small, oc_small, 1), (big, oc_big, 2)):
            Q = synth.queries(7, 0, step, g.B, g.Hq)
            want, outs = _both(gu, g, Q)
            ref = oc.decode_attn(Q)
            gu.assert_attention_close(want, ref, "kvq_decode_attn against the oracle")
            for got in outs:
                assert np.array_equal(got, want), "static-scratch decode differs from kvq_decode_attn"
                gu.assert_attention_close(got, ref, "static-scratch decode against the oracle")
        assert kq.kvq_device_status(big.ctx) == 0 and kq.kvq_device_status(small.ctx) == 0
        # kvq_recover leaves a healthy handle (and the shared array) as it was
        kq.kvq_recover(big.ctx)
        Q = synth.queries(7, 0, 3, big.B, big.Hq)
        want, outs = _both(gu, big, Q)
        assert all(np.array_equal(got, want) for got in outs)
    finally:
        big.close()
        small.close()


def test_static_scratch_entry_rejects_what_does_not_fit(gu, oracle):
    import torch
    from paper_2604_04722_b200 import binding as kq
    g, oc = _filled_cache(gu, oracle, 16, 9, 3, 40, seed=13)
    try:
        Q = synth.queries(7, 0, 0, g.B, g.Hq)
        Qd = gu.dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        kq.kvq_set_splits(g.ctx, 64)                      # 16 * 9 * (64 + 1) = 9360 records > 8192
        assert 16 * 9 * 65 > kq.KVQ_STATIC_MAX_PARTIALS
        with pytest.raises(kq.KvqError) as err:
            kq.kvq_decode_attn_static(g.ctx, 0, Qd, O)
        assert err.value.code == kq.KVQ_ERR_TOO_LARGE
        assert "static scratch" in str(err.value)
        kq.kvq_set_splits(g.ctx, 55)                      # 16 * 9 * 56 = 8064 records fit
        kq.kvq_decode_attn_static(g.ctx, 0, Qd, O)
        want = torch.zeros_like(Qd)
        kq.kvq_decode_attn(g.ctx, 0, Qd, want)
        torch.cuda.synchronize()
        assert np.array_equal(O.cpu().numpy().view(np.uint16), want.cpu().numpy().view(np.uint16)), "55 parts"
        gu.assert_attention_close(O.cpu().numpy().view(np.uint16), oc.decode_attn(Q), "55 parts against the oracle")
    finally:
        g.close()


def test_static_scratch_automatic_plan_fits_the_array(gu, oracle):
    """In automatic mode the planner is told how many records the fixed array holds and only picks plans that
    fit it.  64 * 40 = 2560 units leave room for at most 2 parts per unit (2560 * 3 = 7680 <= 8192 < 2560 * 4):
    the call must run (not KVQ_ERR_TOO_LARGE) and agree with kvq_decode_attn, whose own scratch is larger."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    g, _ = _filled_cache(gu, None, 64, 40, 1, 6000, seed=14)
    try:
        assert 64 * 40 * 4 > kq.KVQ_STATIC_MAX_PARTIALS
        Q = synth.queries(7, 0, 0, g.B, g.Hq)
        Qd = gu.dev(Q.view(np.uint16))
        got, want = torch.full_like(Qd, 0x7e00), torch.zeros_like(Qd)
        kq.kvq_decode_attn_static(g.ctx, 0, Qd, got)
        kq.kvq_decode_attn(g.ctx, 0, Qd, want)
        torch.cuda.synchronize()
        # the two planners may cut differently (another summation order): the attention tolerance applies
        gu.assert_attention_close(got.cpu().numpy().view(np.uint16), want.cpu().numpy().view(np.uint16), "automatic plans")
        kq.kvq_set_splits(g.ctx, 2)                       # the same plan for both: now bit for bit
        kq.kvq_decode_attn(g.ctx, 0, Qd, want)
        got2 = torch.full_like(Qd, 0x7e00)
        kq.kvq_decode_attn_static(g.ctx, 0, Qd, got2)
        kq.kvq_set_splits(g.ctx, 3)                       # 2560 * 4 records do not fit
        with pytest.raises(kq.KvqError) as err:
            kq.kvq_decode_attn_static(g.ctx, 0, Qd, got)
        assert err.value.code == kq.KVQ_ERR_TOO_LARGE
        torch.cuda.synchronize()
        assert np.array_equal(got2.cpu().numpy().view(np.uint16), want.cpu().numpy().view(np.uint16))
        assert kq.kvq_device_status(g.ctx) == 0
    finally:
        g.close()
