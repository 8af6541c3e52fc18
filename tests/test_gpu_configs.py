"""GPU parity on the five benchmark workloads (SmolLM-shaped synthetic caches).

The CUDA path always runs at full size, in the launch configuration the benchmark times.  The
oracle recomputes every sequence of the batch for the attention output (in groups of sequences,
so that its position-ordered cache stays small on the host) and the whole stored form -- every
position: bit-width, (pool, slot), codes, scale / zero-point -- of the sequences named in each
test, bit for bit."""
import numpy as np
import pytest

from paper_2604_04722_b200 import synth

pytestmark = pytest.mark.gpu

STORE_WINDOW = 2048          # positions exported per call when a whole sequence is compared


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


def _compare_whole_store(g, layer, oc, seqs):
    """Every cached position of the sequences `seqs` (rows of `oc` in that order), window by window."""
    n = len(oc)
    for pos0 in range(0, n, STORE_WINDOW):
        m = min(STORE_WINDOW, n - pos0)
        bits, ps, kc, vc, km, vm = g.export(layer, pos0, m)
        sl = slice(pos0, pos0 + m)
        assert np.array_equal(bits[seqs], oc.bits[:, sl]), "bit-widths differ in [%d, %d)" % (pos0, pos0 + m)
        assert np.array_equal(ps[seqs], oc.pool_slot[:, sl]), "(pool, slot) differ in [%d, %d)" % (pos0, pos0 + m)
        assert np.array_equal(km[seqs], oc.km[:, sl]) and np.array_equal(vm[seqs], oc.vm[:, sl]), \
            "scale / zero-point differ in [%d, %d)" % (pos0, pos0 + m)
        assert np.array_equal(kc[seqs], oc.kc[:, sl]), "K codes differ in [%d, %d)" % (pos0, pos0 + m)
        assert np.array_equal(vc[seqs], oc.vc[:, sl]), "V codes differ in [%d, %d)" % (pos0, pos0 + m)


def _compare_all_sequences(gu, oracle, wl, g, layer, K, V, bits, Q, out, store_seqs, group=4, what=""):
    """Attention of EVERY sequence against the oracle, `group` sequences at a time; the whole store of
    the sequences in `store_seqs`."""
    B = K.shape[0]
    for s0 in range(0, B, group):
        seqs = list(range(s0, min(B, s0 + group)))
        oc = _sub_cache(oracle, wl, K, V, bits, seqs)
        gu.assert_attention_close(out[seqs], oc.decode_attn(Q[seqs]), "%s layer %d seqs %s" % (what, layer, seqs))
        mine = [s for s in seqs if s in store_seqs]
        if mine:
            rows = [seqs.index(s) for s in mine]
            sub = oracle.OracleCache(len(mine), wl.q_heads, wl.kv_heads)
            sub.bits, sub.pool_slot = oc.bits[rows], oc.pool_slot[rows]
            sub.kc, sub.vc, sub.km, sub.vm = oc.kc[rows], oc.vc[rows], oc.km[rows], oc.vm[rows]
            _compare_whole_store(g, layer, sub, mine)
        del oc


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


@pytest.mark.parametrize("name,layers", [("cfg2", (0, 29)), ("cfg3", (0, 31))])
def test_cfg2_cfg3_controller_bits_prefill_then_decode_steps(gu, oracle, name, layers):
    """Full-size handle; the checked layers get the full prefill and EVERY decode step of the workload
    (64 and 128), each step appending one controller-decided token per sequence and attending over
    everything cached; at the end the whole store of the checked layers is compared."""
    wl = synth.CONFIGS[name]
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)
    B, steps = wl.batch, wl.decode_steps
    feats = synth.features_batch(wl.seed, B, 0, wl.context)
    want_bits, want_logits, gap = oracle.select_bits(feats, wl.hidden, *cw.as_tuple())
    with gu.GpuCache(wl.layers, B, wl.q_heads, wl.kv_heads, wl.max_ctx) as g:
        g.set_controller(cw)
        got_bits, _ = g.select_bits(feats)
        near = gu.compare_decisions(got_bits, want_bits, want_logits, gap, "%s prefill decisions" % name)
        assert all(r[3] == r[4] for r in near), "a near tie was decided differently: %s" % near[:3]
        ocs = {}
        for layer in layers:
            K, V = synth.kv_batch(wl.seed, layer, B, 0, wl.context, wl.kv_heads)
            oc = oracle.OracleCache(B, wl.q_heads, wl.kv_heads)
            oc.append(K, V, want_bits)
            assert np.array_equal(g.append_fused(layer, K, V, feats), want_bits)
            ocs[layer] = oc
        step_feats = np.concatenate([synth.features_batch(wl.seed, B, wl.context + s, 1) for s in range(steps)], axis=1)
        sb, sl, sg = oracle.select_bits(step_feats, wl.hidden, *cw.as_tuple())
        got_steps = np.zeros_like(sb)
        for step in range(steps):
            t0 = wl.context + step
            f1 = step_feats[:, step:step + 1]
            b1 = sb[:, step:step + 1]
            for layer in layers:
                K, V = synth.kv_batch(wl.seed, layer, B, t0, 1, wl.kv_heads)
                Q = synth.queries(wl.seed, layer, step, B, wl.q_heads)
                ocs[layer].append(K, V, b1)
                got_steps[:, step:step + 1] = g.append_fused(layer, K, V, f1)
                gu.assert_attention_close(g.decode(layer, Q), ocs[layer].decode_attn(Q),
                                          "%s layer %d step %d" % (name, layer, step))
        near = gu.compare_decisions(got_steps, sb, sl, sg, "%s decode-step decisions" % name)
        assert all(r[3] == r[4] for r in near)         # the stores below were built from the oracle's decisions
        for layer in layers:
            gu.assert_store_equals_oracle(g, layer, ocs[layer])


@pytest.mark.parametrize("variant", ["runs", 2, 4, 8, 16])
def test_cfg4_runs_and_static_baselines(gu, oracle, variant):
    """Two of the 24 layers (their own seeded K/V) at full batch and context; the handle is sized for one
    layer so that the five variants fit comfortably, and is reset between the two.  All 16 sequences are
    checked for attention, the whole store of sequences 0 and 15."""
    wl = synth.CONFIGS["cfg4"]
    B = wl.batch
    from paper_2604_04722_b200 import binding as kq
    with gu.GpuCache(1, B, wl.q_heads, wl.kv_heads, wl.max_ctx) as g:
        for layer in (7, 20):
            K, V = synth.kv_batch(wl.seed, layer, B, 0, wl.context, wl.kv_heads)
            if variant == "runs":
                bits = np.stack([synth.workload_bits(wl, b, 0, wl.context) for b in range(B)])
            else:
                bits = np.full((B, wl.context), variant, np.uint8)
            Q = synth.queries(wl.seed, layer, 0, B, wl.q_heads)
            kq.kvq_reset(g.ctx)
            g.append(0, K, V, bits)
            out = g.decode(0, Q)
            _compare_all_sequences(gu, oracle, wl, g, 0, K, V, bits, Q, out, store_seqs=(0, 15),
                                   what="cfg4 %s (data of layer %d)" % (variant, layer))
            assert kq.kvq_device_status(g.ctx) == 0


def test_cfg5_stress_prefill_through_controller_then_mixed_decode(gu, oracle):
    """Phase 1: prefill all 32768 tokens per sequence with controller-decided bits.  Phase 2: reset,
    re-append with the stated i.i.d. mix, decode.  Both phases: attention of all 16 sequences, the whole
    store (all 32768 positions) of sequences 5 and 12."""
    wl = synth.CONFIGS["cfg5"]
    B = wl.batch
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)
    K, V = synth.kv_batch(wl.seed, 0, B, 0, wl.context, wl.kv_heads)
    Q = synth.queries(wl.seed, 0, 0, B, wl.q_heads)
    feats = synth.features_batch(wl.seed, B, 0, wl.context)
    from paper_2604_04722_b200 import binding as kq
    with gu.GpuCache(1, B, wl.q_heads, wl.kv_heads, wl.max_ctx) as g:
        g.set_controller(cw)
        ctl_bits, ctl_logits, gap = oracle.select_bits(feats, wl.hidden, *cw.as_tuple())
        got = g.append_fused(0, K, V, feats)
        near = gu.compare_decisions(got, ctl_bits, ctl_logits, gap, "cfg5 prefill decisions")
        assert all(r[3] == r[4] for r in near)
        _compare_all_sequences(gu, oracle, wl, g, 0, K, V, ctl_bits, Q, g.decode(0, Q), store_seqs=(5, 12),
                               what="cfg5 controller bits")
        kq.kvq_reset(g.ctx)
        bits = np.stack([synth.workload_bits(wl, b, 0, wl.context) for b in range(B)])
        g.append(0, K, V, bits)
        _compare_all_sequences(gu, oracle, wl, g, 0, K, V, bits, Q, g.decode(0, Q), store_seqs=(5, 12),
                               what="cfg5 iid mix")
        assert kq.kvq_device_status(g.ctx) == 0
