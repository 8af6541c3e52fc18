"""Ragged batches: sequences of one layer append different numbers of tokens per call and end up with
different lengths.  Every sequence is checked against its own single-sequence oracle cache."""
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
    K = (rng.standard_normal((B, n, H, 64)) * 1.5).astype(np.float16)
    V = (rng.standard_normal((B, n, H, 64)) * 1.5).astype(np.float16)
    return K, V


def test_ragged_appends_uniform_appends_and_steps_on_one_layer(gu, oracle):
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(31)
    B, Hq, H, max_ctx = 3, 6, 2, 900
    cw = synth.controller_weights(322, 32)
    ocs = [oracle.OracleCache(1, Hq, H) for _ in range(B)]

    def oracle_add(b, K, V, bits):
        if K.shape[0]:
            ocs[b].append(K[None], V[None], bits[None])

    with gu.GpuCache(1, B, Hq, H, max_ctx) as g:
        g.set_controller(cw)
        # 1. ragged, bit-widths given, several chunks for sequence 0, nothing for sequence 2
        lens = [700, 300, 0]
        K, V = _kv(rng, B, 700, H)
        bits = BITS[rng.choice(4, size=(B, 700), p=[.4, .3, .2, .1])]
        kq.kvq_append_ragged(g.ctx, 0, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits), None, 700, lens)
        for b in range(B):
            oracle_add(b, K[b, :lens[b]], V[b, :lens[b]], bits[b, :lens[b]])
        assert kq.kvq_seq_lens(g.ctx, 0, B).tolist() == lens and kq.kvq_seq_len(g.ctx, 0) == 700
        # 2. a uniform append on the now ragged layer
        K, V = _kv(rng, B, 5, H)
        bits = BITS[rng.choice(4, size=(B, 5))]
        g.append(0, K, V, bits)
        for b in range(B):
            oracle_add(b, K[b], V[b], bits[b])
        # 3. ragged with the controller deciding inside the launch
        lens3 = [3, 40, 17]
        K, V = _kv(rng, B, 40, H)
        feats = synth.features_batch(9, B, 0, 40)
        want_bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
        got_bits = torch.zeros((B, 40), dtype=torch.uint8, device=gu.DEV)
        kq.kvq_append_ragged(g.ctx, 0, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), None,
                             gu.dev(feats.astype(np.float32)), 40, lens3, got_bits)
        torch.cuda.synchronize()
        for b in range(B):
            assert np.array_equal(got_bits.cpu().numpy()[b, :lens3[b]], want_bits[b, :lens3[b]])
            oracle_add(b, K[b, :lens3[b]], V[b, :lens3[b]], want_bits[b, :lens3[b]])
        # 4. decode steps: one token for everybody, then attend
        for step in range(3):
            K, V = _kv(rng, B, 1, H)
            bits = BITS[rng.choice(4, size=(B, 1))]
            g.append(0, K, V, bits)
            for b in range(B):
                oracle_add(b, K[b], V[b], bits[b])
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            out = g.decode(0, Q)
            for b in range(B):
                gu.assert_attention_close(out[b:b + 1], ocs[b].decode_attn(Q[b:b + 1]), "step %d seq %d" % (step, b))
        want_lens = [len(oc) for oc in ocs]
        assert kq.kvq_seq_lens(g.ctx, 0, B).tolist() == want_lens == [711, 348, 25]
        # the store, token by token at a sample of positions of every sequence
        for b in range(B):
            for pos in sorted({0, 1, 4, 5, want_lens[b] // 2, want_lens[b] - 4, want_lens[b] - 1}):
                bt, ps, kc, vc, km, vm = kq.kvq_export_token(g.ctx, 0, b, pos, H)
                oc = ocs[b]
                assert bt == int(oc.bits[0, pos]) and ps == int(oc.pool_slot[0, pos]), (b, pos)
                assert np.array_equal(kc, oc.kc[0, pos]) and np.array_equal(vc, oc.vc[0, pos]), (b, pos)
                assert np.array_equal(km, oc.km[0, pos]) and np.array_equal(vm, oc.vm[0, pos]), (b, pos)
        # causal rows of the last three positions of every sequence
        T = 3
        Q = rng.standard_normal((B, T, Hq, 64)).astype(np.float16)
        Qd = gu.dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        kq.kvq_attend_last(g.ctx, 0, Qd, O, T)
        torch.cuda.synchronize()
        got = O.cpu().numpy().view(np.uint16)
        for b in range(B):
            gu.assert_attention_close(got[b:b + 1], ocs[b].attend_last(Q[b:b + 1]), "causal rows seq %d" % b)
        # limits: positions past the shortest sequence, lengths out of range, capacity of one sequence
        assert kq.lib().kvq_export_range(g.ctx, 0, 20, 10, None, None, None, None, None, None, None) == kq.KVQ_ERR_ARG
        Kd = gu.dev(np.zeros((B, 200, H, 64), np.uint16))
        bd = gu.dev(np.full((B, 200), 4, np.uint8))
        bad = np.array([0, 201, 0], np.int32)
        assert kq.lib().kvq_append_ragged(g.ctx, 0, Kd.data_ptr(), Kd.data_ptr(), bd.data_ptr(), None, 200,
                                          bad.ctypes.data, None, None) == kq.KVQ_ERR_ARG
        over = np.array([200, 0, 0], np.int32)                        # 711 + 200 > 900
        assert kq.lib().kvq_append_ragged(g.ctx, 0, Kd.data_ptr(), Kd.data_ptr(), bd.data_ptr(), None, 200,
                                          over.ctypes.data, None, None) == kq.KVQ_ERR_CAPACITY
        assert kq.kvq_device_status(g.ctx) == 0


def test_a_sequence_without_tokens_gets_a_zero_row(gu, oracle):
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(32)
    B, Hq, H = 2, 4, 2
    K, V = _kv(rng, B, 50, H)
    bits = BITS[rng.choice(4, size=(B, 50))]
    with gu.GpuCache(1, B, Hq, H, 64) as g:
        kq.kvq_append_ragged(g.ctx, 0, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits), None, 50, [50, 0])
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        out = g.decode(0, Q)
        oc = oracle.OracleCache(1, Hq, H)
        oc.append(K[:1], V[:1], bits[:1])
        gu.assert_attention_close(out[:1], oc.decode_attn(Q[:1]), "the filled sequence")
        assert not out[1].any()
