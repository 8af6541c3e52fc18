"""kvq_decode_attn_static: decode attention for callers that must not allocate.

A serving loop under a "no allocation after start-up" rule, or a plug-in living inside a
process whose device memory belongs to another allocator, cannot let a library reserve scratch
for it.  This entry point keeps the split-attention partials in a fixed array inside the library
image instead, so the call itself performs no allocation.  The test drives it through the C ABI
and checks that it returns what kvq_decode_attn returns -- twice in a row, because the array is
shared by all calls and keeps the previous call's contents, and once more on a different cache
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


def _filled_cache(gu, batch, q_heads, kv_heads, n, seed):
    K, V = synth.kv_batch(seed, 0, batch, 0, n, kv_heads)
    bits = np.stack([synth.bits_iid(seed, b, 0, n, (0.4, 0.3, 0.2, 0.1)) for b in range(batch)])
    g = gu.GpuCache(1, batch, q_heads, kv_heads, n)
    g.append(0, K, V, bits)
    return g


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


def test_static_scratch_entry_matches_the_allocating_one_twice_in_a_row(gu):
    from paper_2604_04722_b200 import binding as kq
    big = _filled_cache(gu, 4, 6, 2, 3000, seed=11)       # several splits, ragged last tiles
    small = _filled_cache(gu, 2, 3, 3, 70, seed=12)       # a smaller problem afterwards
    try:
        for g, step in ((big, 0), (small, 1), (big, 2)):
            Q = synth.queries(7, 0, step, g.B, g.Hq)
            want, outs = _both(gu, g, Q)
            for got in outs:
                gu.assert_attention_close(got, want, "static-scratch decode")
        assert kq.kvq_device_status(big.ctx) == 0 and kq.kvq_device_status(small.ctx) == 0
    finally:
        big.close()
        small.close()


def test_static_scratch_entry_rejects_what_does_not_fit(gu):
    import torch
    from paper_2604_04722_b200 import binding as kq
    g = _filled_cache(gu, 16, 9, 3, 40, seed=13)
    try:
        Qd = gu.dev(synth.queries(7, 0, 0, g.B, g.Hq).view(np.uint16))
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
        gu.assert_attention_close(O.cpu().numpy().view(np.uint16), want.cpu().numpy().view(np.uint16), "55 parts")
    finally:
        g.close()
