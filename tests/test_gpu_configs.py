"""GPU parity on the five benchmark workloads (SmolLM-shaped synthetic caches).

Small workloads are compared in full; for the large ones the CUDA path runs at full size, in the
launch configuration the benchmark times, and the oracle recomputes a sample of sequences
(every head of those sequences, every cached token)."""
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


def _sub_cache(oracle, wl, K, V, bits, seqs):
    oc = oracle.OracleCache(len(seqs), wl.q_heads, wl.kv_heads)
    oc.append(K[seqs], V[seqs], bits[seqs])
    return oc


def _compare_sampled(gu, g, layer, oc, seqs, Q, out, n_check_store=64):
    """Attention of the sampled sequences, and the store rows of a window at both ends."""
    want = oc.decode_attn(Q[seqs])
    gu.assert_attention_close(out[seqs], want, "layer %d seqs %s" % (layer, seqs))
    n = len(oc)
    for pos0 in sorted({0, max(0, n - n_check_store)}):
        m = min(n_check_store, n - pos0)
        bits, ps, kc, vc, km, vm = g.export(layer, pos0, m)
        sl = slice(pos0, pos0 + m)
        assert np.array_equal(bits[seqs], oc.bits[:, sl])
        assert np.array_equal(ps[seqs], oc.pool_slot[:, sl])
        assert np.array_equal(kc[seqs], oc.kc[:, sl]) and np.array_equal(vc[seqs], oc.vc[:, sl])
        assert np.array_equal(km[seqs], oc.km[:, sl]) and np.array_equal(vm[seqs], oc.vm[:, sl])


def test_cfg1_single_layer_decode_step(gu, oracle):
    wl = synth.CONFIGS["cfg1"]
    K, V = synth.kv_batch(wl.seed, 0, wl.batch, 0, wl.context, wl.kv_heads)
    bits = np.stack([synth.workload_bits(wl, b, 0, wl.context) for b in range(wl.batch)])
    Q = synth.queries(wl.seed, 0, 0, wl.batch, wl.q_heads)
    oc = oracle.OracleCache(wl.batch, wl.q_heads, wl.kv_heads)
    oc.append(K, V, bits)
    with gu.GpuCache(wl.layers, wl.batch, wl.q_heads, wl.kv_heads, wl.max_ctx) as g:
        g.append(0, K, V, bits)
        gu.assert_store_equals_oracle(g, 0, oc)
        gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "cfg1")


@pytest.mark.parametrize("name,layers,steps", [("cfg2", (0, 29), 64), ("cfg3", (0, 31), 12)])
def test_cfg2_cfg3_controller_bits_prefill_then_decode_steps(gu, oracle, name, layers, steps):
    """Full-size handle; the checked layers get the full prefill and the decode steps, each step
    appending one controller-decided token per sequence and attending over everything cached."""
    wl = synth.CONFIGS[name]
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)
    B = wl.batch
    feats = synth.features_batch(wl.seed, B, 0, wl.context)
    want_bits, _, gap = oracle.select_bits(feats, wl.hidden, *cw.as_tuple())
    with gu.GpuCache(wl.layers, B, wl.q_heads, wl.kv_heads, wl.max_ctx) as g:
        g.set_controller(cw)
        got_bits, _ = g.select_bits(feats)
        assert np.array_equal(got_bits, want_bits), "near ties: %d" % int((gap < 1e-5).sum())
        ocs = {}
        for layer in layers:
            K, V = synth.kv_batch(wl.seed, layer, B, 0, wl.context, wl.kv_heads)
            oc = oracle.OracleCache(B, wl.q_heads, wl.kv_heads)
            oc.append(K, V, want_bits)
            assert np.array_equal(g.append_fused(layer, K, V, feats), want_bits)
            ocs[layer] = oc
        for step in range(steps):
            t0 = wl.context + step
            f1 = synth.features_batch(wl.seed, B, t0, 1)
            b1, _, _ = oracle.select_bits(f1, wl.hidden, *cw.as_tuple())
            for layer in layers:
                K, V = synth.kv_batch(wl.seed, layer, B, t0, 1, wl.kv_heads)
                Q = synth.queries(wl.seed, layer, step, B, wl.q_heads)
                ocs[layer].append(K, V, b1)
                assert np.array_equal(g.append_fused(layer, K, V, f1), b1)
                gu.assert_attention_close(g.decode(layer, Q), ocs[layer].decode_attn(Q),
                                          "%s layer %d step %d" % (name, layer, step))
        for layer in layers:
            gu.assert_store_equals_oracle(g, layer, ocs[layer])


@pytest.mark.parametrize("variant", ["runs", 2, 4, 8, 16])
def test_cfg4_runs_and_static_baselines(gu, oracle, variant):
    """One of the 24 layers at full batch/context (the handle is sized for one layer so that the
    five variants fit comfortably); sampled sequences 0 and 15 against the oracle."""
    wl = synth.CONFIGS["cfg4"]
    B, layer, seqs = wl.batch, 7, [0, 15]
    K, V = synth.kv_batch(wl.seed, layer, B, 0, wl.context, wl.kv_heads)
    if variant == "runs":
        bits = np.stack([synth.workload_bits(wl, b, 0, wl.context) for b in range(B)])
    else:
        bits = np.full((B, wl.context), variant, np.uint8)
    Q = synth.queries(wl.seed, layer, 0, B, wl.q_heads)
    oc = _sub_cache(oracle, wl, K, V, bits, seqs)
    with gu.GpuCache(1, B, wl.q_heads, wl.kv_heads, wl.max_ctx) as g:
        g.append(0, K, V, bits)
        out = g.decode(0, Q)
        _compare_sampled(gu, g, 0, oc, seqs, Q, out)


def test_cfg5_stress_prefill_through_controller_then_mixed_decode(gu, oracle):
    """Phase 1: prefill all 32768 tokens per sequence with controller-decided bits.  Phase 2:
    reset, re-append with the stated i.i.d. mix, decode.  Sampled sequence: 5."""
    wl = synth.CONFIGS["cfg5"]
    B, seqs = wl.batch, [5]
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)
    K, V = synth.kv_batch(wl.seed, 0, B, 0, wl.context, wl.kv_heads)
    Q = synth.queries(wl.seed, 0, 0, B, wl.q_heads)
    feats = synth.features_batch(wl.seed, B, 0, wl.context)
    from paper_2604_04722_b200 import binding as kq
    with gu.GpuCache(1, B, wl.q_heads, wl.kv_heads, wl.max_ctx) as g:
        g.set_controller(cw)
        ctl_bits, _, _ = oracle.select_bits(feats[seqs], wl.hidden, *cw.as_tuple())
        got = g.append_fused(0, K, V, feats)
        assert np.array_equal(got[seqs], ctl_bits)
        oc = oracle.OracleCache(len(seqs), wl.q_heads, wl.kv_heads)
        oc.append(K[seqs], V[seqs], ctl_bits)
        _compare_sampled(gu, g, 0, oc, seqs, Q, g.decode(0, Q))
        kq.kvq_reset(g.ctx)
        bits = np.stack([synth.workload_bits(wl, b, 0, wl.context) for b in range(B)])
        g.append(0, K, V, bits)
        oc = _sub_cache(oracle, wl, K, V, bits, seqs)
        _compare_sampled(gu, g, 0, oc, seqs, Q, g.decode(0, Q))
