"""Prefill appends with 512-token slot-assignment chunks (the size long prefills pick on their own), forced on
small shapes so that every path is compared with the oracle token by token: bit-widths given and decided by
the controller, ragged batches, grouped scales, chunk ends that fall inside a tile, and a second append that
continues partly filled tiles."""
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


def _kv(rng, B, n, H):
    K = (rng.standard_normal((B, n, H, 64)) * 2).astype(np.float16)
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    return K, V


def test_chunk_size_values(gu):
    from paper_2604_04722_b200 import binding as kq
    with gu.GpuCache(1, 1, 1, 1, 16) as g:
        for ok in (0, 256, 512, 0):
            kq.kvq_set_append_chunk(g.ctx, ok)
        for bad in (1, 128, 1024, -256):
            assert kq.lib().kvq_set_append_chunk(g.ctx, bad) == kq.KVQ_ERR_ARG


@pytest.mark.parametrize("groups", [1, 2])
@pytest.mark.parametrize("sizes", [[1300], [513, 511, 700], [257, 1, 1030]])
def test_given_bits_and_controller_bits_with_512_token_chunks(gu, oracle, groups, sizes):
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(sum(sizes) + groups)
    B, Hq, H = 2, 6, 3
    cw = synth.controller_weights(322, 32)
    oc = oracle.OracleCache(B, Hq, H) if groups == 1 else oracle.GroupedOracleCache(B, Hq, H, 2)
    with gu.GpuCache(1, B, Hq, H, 2 * sum(sizes) + 8, scale_groups=groups) as g:
        g.set_controller(cw)
        kq.kvq_set_append_chunk(g.ctx, 512)
        pos = 0
        for fused in (False, True):
            for n in sizes:
                K, V = _kv(rng, B, n, H)
                if fused:
                    feats = synth.features_batch(7, B, pos, n)
                    bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
                    assert np.array_equal(g.append_fused(0, K, V, feats), bits)
                else:
                    bits = BITS[rng.choice(4, size=(B, n), p=[.45, .3, .2, .05])]
                    g.append(0, K, V, bits)
                oc.append(K, V, bits)
                pos += n
        gu.assert_store_equals_oracle(g, 0, oc)
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "after the appends")
        counts, _, _ = kq.kvq_stats(g.ctx, 0, B)
        assert np.array_equal(counts, oc.counts)


def test_ragged_prefill_with_512_token_chunks(gu, oracle):
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(77)
    B, Hq, H, n = 3, 4, 2, 1100
    lens = [1100, 515, 0]
    K, V = _kv(rng, B, n, H)
    bits = BITS[rng.choice(4, size=(B, n), p=[.4, .3, .2, .1])]
    ocs = [oracle.OracleCache(1, Hq, H) for _ in range(B)]
    with gu.GpuCache(1, B, Hq, H, n + 600) as g:
        kq.kvq_set_append_chunk(g.ctx, 512)
        kq.kvq_append_ragged(g.ctx, 0, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits), None, n, lens)
        lens2 = [0, 600, 300]
        K2, V2 = _kv(rng, B, 600, H)
        bits2 = BITS[rng.choice(4, size=(B, 600))]
        kq.kvq_append_ragged(g.ctx, 0, gu.dev(K2.view(np.uint16)), gu.dev(V2.view(np.uint16)), gu.dev(bits2), None, 600, lens2)
        for b in range(B):
            if lens[b]:
                ocs[b].append(K[b:b + 1, :lens[b]], V[b:b + 1, :lens[b]], bits[b:b + 1, :lens[b]])
            if lens2[b]:
                ocs[b].append(K2[b:b + 1, :lens2[b]], V2[b:b + 1, :lens2[b]], bits2[b:b + 1, :lens2[b]])
        assert kq.kvq_seq_lens(g.ctx, 0, B).tolist() == [1100, 1115, 300]
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        out = g.decode(0, Q)
        for b in range(B):
            gu.assert_attention_close(out[b:b + 1], ocs[b].decode_attn(Q[b:b + 1]), "sequence %d" % b)
