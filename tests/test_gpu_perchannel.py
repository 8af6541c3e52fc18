"""Per-channel keys (kvq_create_perchannel) against the oracle's PerChannelKCache: the stored form bit for bit
(value codes and pairs, key codes of complete windows, fp16 key rows of open windows, the per-channel pairs of
every complete window), attention within the usual tolerance."""
import numpy as np
import pytest

from paper_2604_04722_b200 import synth

pytestmark = pytest.mark.gpu

BITS = np.array([2, 4, 8, 16], np.uint8)


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_04722_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _kv(rng, B, n, H, scale=1.0):
    K = (rng.standard_normal((B, n, H, 64)) * scale).astype(np.float16)
    K[..., 5] *= 8                                        # an outlier channel, the case per-channel scales are for
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    return K, V


def assert_store_equals(gu, g, oc, layer=0):
    from paper_2604_04722_b200 import binding as kq
    n = len(oc)
    bits, ps, kc, vc, km, vm = g.export(layer, 0, n)
    state, want_kc, _, chan = oc.key_state()
    assert np.array_equal(bits, oc.bits) and np.array_equal(ps, oc.pool_slot)
    assert np.array_equal(vm, oc.vm), "value scale / zero-point differ"
    assert np.array_equal(vc, oc.vc), "value codes differ"
    assert not km.any()
    bad = np.argwhere((kc != want_kc).any(axis=-1))
    assert bad.size == 0, "key rows differ first at (b, pos, head) %s (state %d, bits %d)" % (
        bad[0], state[tuple(bad[0])], oc.bits[bad[0][0], bad[0][1]])
    for (b, h, bt, w), want in chan.items():
        got = kq.kvq_export_k_channels(g.ctx, layer, b, h, bt, w)
        assert np.array_equal(got, want), "channel pairs of window %d (b %d head %d, %d bits) differ" % (w, b, h, bt)
    return len(chan)


@pytest.mark.parametrize("n,mix", [(16, (1, 0, 0, 0)), (300, (.4, .3, .2, .1)), (700, (.5, .3, .15, .05)), (1500, (0, 1, 0, 0))])
def test_prefill_store_and_attention(gu, oracle, n, mix):
    rng = np.random.default_rng(n)
    B, Hq, H = 2, 6, 2
    K, V = _kv(rng, B, n, H, 1.5)
    bits = BITS[rng.choice(4, size=(B, n), p=mix)]
    oc = oracle.PerChannelKCache(B, Hq, H)
    oc.append(K, V, bits)
    with gu.GpuCache(1, B, Hq, H, n + 8, k_per_channel=True) as g:
        g.append(0, K, V, bits)
        assert assert_store_equals(gu, g, oc) > 0
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "prefill n=%d" % n)


def test_windows_fill_across_calls_and_token_steps(gu, oracle):
    """A prefill, token steps (each may complete a window of its precision), small and multi-chunk appends: after
    every phase the store and the attention agree with the oracle."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(3)
    B, Hq, H = 3, 9, 3
    sizes = [100] + [1] * 45 + [37] + [1] * 20 + [300, 1, 1, 1]
    oc = oracle.PerChannelKCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, sum(sizes), k_per_channel=True) as g:
        for k, n in enumerate(sizes):
            K, V = _kv(rng, B, n, H)
            bits = BITS[rng.choice(4, size=(B, n), p=[.4, .3, .2, .1])]
            oc.append(K, V, bits)
            g.append(0, K, V, bits)
            if n > 1 or k % 9 == 0 or k == len(sizes) - 1:
                assert_store_equals(gu, g, oc)
                Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
                for splits in (0, 1, 5):
                    kq.kvq_set_splits(g.ctx, splits)
                    gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "after call %d, splits %d" % (k, splits))
        assert kq.kvq_device_status(g.ctx) == 0


def test_controller_inside_and_snapshot(gu, oracle):
    """kvq_append_fused on this layout (prefill and token steps), several arena blocks per stream, and a snapshot
    taken with open windows that continues in a fresh handle."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(8)
    cw = synth.controller_weights(322, 32)
    B, Hq, H, n = 2, 4, 4, 2100
    feats = synth.features_batch(4, B, 0, n + 30)
    want_bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
    K, V = _kv(rng, B, n + 30, H)
    oc = oracle.PerChannelKCache(B, Hq, H)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    with gu.GpuCache(1, B, Hq, H, n + 30, k_per_channel=True) as g:
        g.set_controller(cw)
        assert np.array_equal(g.append_fused(0, K[:, :n], V[:, :n], feats[:, :n]), want_bits[:, :n])
        oc.append(K[:, :n], V[:, :n], want_bits[:, :n])
        for t in range(n, n + 10):
            assert np.array_equal(g.append_fused(0, K[:, t:t + 1], V[:, t:t + 1], feats[:, t:t + 1]), want_bits[:, t:t + 1])
            oc.append(K[:, t:t + 1], V[:, t:t + 1], want_bits[:, t:t + 1])
        assert_store_equals(gu, g, oc)
        gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "fused")
        blob = kq.kvq_save_state(g.ctx)
    with gu.GpuCache(1, B, Hq, H, n + 30, k_per_channel=True) as g2:
        g2.set_controller(cw)
        kq.kvq_load_state(g2.ctx, blob)
        for t in range(n + 10, n + 30):
            g2.append_fused(0, K[:, t:t + 1], V[:, t:t + 1], feats[:, t:t + 1])
            oc.append(K[:, t:t + 1], V[:, t:t + 1], want_bits[:, t:t + 1])
        assert_store_equals(gu, g2, oc)
        gu.assert_attention_close(g2.decode(0, Q), oc.decode_attn(Q), "after the snapshot")
        import torch
        Qd = gu.dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        with pytest.raises(kq.KvqError):
            kq.kvq_attend_last(g2.ctx, 0, torch.stack([Qd, Qd], dim=1).contiguous(), torch.zeros((B, 2, Hq, 64), dtype=Qd.dtype, device=Qd.device), 2)


def test_ragged_appends_and_the_static_scratch_entry(gu, oracle):
    """Sequences that grow by different amounts (one oracle cache per sequence), and kvq_decode_attn_static on this
    layout: bit for bit what kvq_decode_attn returns."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(21)
    B, Hq, H, n_max = 3, 4, 2, 90
    ocs = [oracle.PerChannelKCache(1, Hq, H) for _ in range(B)]
    with gu.GpuCache(1, B, Hq, H, 4 * n_max, k_per_channel=True) as g:
        for call in range(4):
            K, V = _kv(rng, B, n_max, H)
            bits = BITS[rng.choice(4, size=(B, n_max), p=[.4, .3, .2, .1])]
            lens = rng.integers(1, n_max + 1, size=B)
            kq.kvq_append_ragged(g.ctx, 0, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits), None, n_max, lens)
            for b in range(B):
                ocs[b].append(K[b:b + 1, :lens[b]], V[b:b + 1, :lens[b]], bits[b:b + 1, :lens[b]])
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        out = g.decode(0, Q)
        for b in range(B):
            gu.assert_attention_close(out[b:b + 1], ocs[b].decode_attn(Q[b:b + 1]), "sequence %d" % b)
        Qd = gu.dev(Q.view(np.uint16))
        got = torch.full_like(Qd, 0x7e00)
        kq.kvq_decode_attn_static(g.ctx, 0, Qd, got)
        torch.cuda.synchronize()
        assert np.array_equal(got.cpu().numpy().view(np.uint16), out)
        assert kq.kvq_device_status(g.ctx) == 0
