"""GPU parity of kvq_decode_step: one decode step (controller decision, quantize-append of one
token per sequence, attention over everything cached, Eq. 19-24, Eq. 4, Eq. 5) against the
oracle, step by step.  With keys quantized per token the step is one launch (the attending warps
add the step's token themselves from its fp16 rows); per-channel keys run the two kernels of
kvq_append_fused + kvq_decode_attn behind the same call.  Both are compared with the
oracle the same way: decisions and the whole store bit for bit, the attention output of EVERY
step within the attention tolerance."""
import numpy as np
import pytest

from paper_2604_04722_b200 import synth

pytestmark = pytest.mark.gpu

BITS = np.array([2, 4, 8, 16], dtype=np.uint8)


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
    V = (rng.standard_normal((B, n, H, 64)) * scale).astype(np.float16)
    return K, V


def _step(gu, g, layer, feats, K, V, Q):
    """kvq_decode_step through the binding; returns (decisions [B], output [B][Hq][64] as uint16)."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    fd, Kd, Vd = gu.dev(feats.astype(np.float32)), gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16))
    Qd = gu.dev(Q.view(np.uint16))
    O = torch.zeros_like(Qd)
    bits = torch.zeros(feats.shape[0], dtype=torch.uint8, device=gu.DEV)
    kq.kvq_decode_step(g.ctx, layer, fd, Kd, Vd, Qd, O, bits)
    torch.cuda.synchronize()
    return bits.cpu().numpy(), O.cpu().numpy().view(np.uint16)


def _run_steps(gu, oracle, g, oc, cw, rng, B, Hq, H, steps, what, feat_seed=3, kscale=1.0, layer=0, first_pos=0):
    from paper_2604_04722_b200 import binding as kq
    feats = synth.features_batch(feat_seed, B, first_pos, steps)
    want_bits, want_logits, gap = oracle.select_bits(feats, cw.hidden, *cw.as_tuple())
    got_bits = np.zeros_like(want_bits)
    launches0 = kq.kvq_launch_count(g.ctx)
    for s in range(steps):
        K, V = _kv(rng, B, 1, H, kscale)
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        oc.append(K, V, want_bits[:, s:s + 1])
        got_bits[:, s], out = _step(gu, g, layer, feats[:, s], K, V, Q)
        gu.assert_attention_close(out, oc.decode_attn(Q), "%s, step %d" % (what, s))
    near = gu.compare_decisions(got_bits, want_bits, want_logits, gap, what)
    assert all(r[3] == r[4] for r in near)      # the oracle's store below was built from the oracle's decisions
    assert kq.kvq_device_status(g.ctx) == 0
    return kq.kvq_launch_count(g.ctx) - launches0


@pytest.mark.parametrize("B,Hq,H", [(3, 6, 2), (1, 9, 3), (2, 20, 20)])
def test_steps_from_an_empty_cache_take_one_launch_each(gu, oracle, B, Hq, H):
    """From nothing cached: the first step attends over its own token only.  70 steps cross several tiles of every
    pool; 20 KV heads need two storing warps per sequence."""
    rng = np.random.default_rng(100 + B)
    cw = synth.controller_weights(322, 32)
    steps = 70
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, steps) as g:
        g.set_controller(cw)
        launches = _run_steps(gu, oracle, g, oc, cw, rng, B, Hq, H, steps, "step from empty B=%d" % B)
        assert launches == steps                 # one kernel per step
        gu.assert_store_equals_oracle(g, 0, oc)
        assert len(set(oc.bits.ravel().tolist())) >= 3


@pytest.mark.parametrize("splits", [0, 1, 2, 7, 16])
def test_steps_after_a_prefill_for_every_way_of_cutting_the_work(gu, oracle, splits):
    """Prefill of mixed precision, then steps; the split count decides whether the parts of a unit meet inside
    their CTA (1, 2, 16, automatic) or through partial records (7): the token is added by the unit's last part."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(200 + splits)
    cw = synth.controller_weights(98, 32)
    B, Hq, H, n, steps = 2, 9, 3, 777, 24
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(2, B, Hq, H, n + steps) as g:
        g.set_controller(cw)
        kq.kvq_set_splits(g.ctx, splits)
        K, V = _kv(rng, B, n, H, 1.5)
        bits = BITS[rng.choice(4, size=(B, n))]
        oc.append(K, V, bits)
        g.append(1, K, V, bits)
        launches = _run_steps(gu, oracle, g, oc, cw, rng, B, Hq, H, steps, "step after prefill, splits=%d" % splits,
                              kscale=1.5, layer=1, first_pos=n)
        assert launches == steps
        gu.assert_store_equals_oracle(g, 1, oc)


def test_steps_that_open_new_blocks_and_new_tiles(gu, oracle):
    """All tokens in one class (a controller whose biases decide): the 2-bit stream of a sequence fills its first
    64 KB block (100 tiles of 16 slots) during the steps and goes on in a second one."""
    rng = np.random.default_rng(5)
    H32 = 32
    z = np.zeros
    cw = synth.ControllerWeights(H32, z((H32, 4), np.float32), z(H32, np.float32), z((H32, H32), np.float32),
                                 z(H32, np.float32), z((4, H32), np.float32), np.array([1, 0, 0, 0], np.float32))
    B, Hq, H = 1, 2, 1
    n = 100 * 16 - 5
    steps = 12
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, n + steps) as g:
        g.set_controller(cw)
        K, V = _kv(rng, B, n, H)
        bits = np.full((B, n), 2, np.uint8)
        oc.append(K, V, bits)
        g.append(0, K, V, bits)
        _run_steps(gu, oracle, g, oc, cw, rng, B, Hq, H, steps, "steps across a block border", first_pos=n)
        assert set(oc.bits.ravel().tolist()) == {2}
        gu.assert_store_equals_oracle(g, 0, oc, pos0=n - 40, n=40 + steps)


@pytest.mark.parametrize("splits", [0, 3, 4])
def test_steps_on_a_long_cache_in_the_bandwidth_geometry(gu, oracle, splits):
    """40 000 cached tokens per sequence: the launch takes the geometry of four-warp CTAs; parts of a unit meet
    through partial records (automatic plan, 3) or inside their CTA (4)."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(300 + splits)
    cw = synth.controller_weights(322, 32)
    B, Hq, H, n, steps = 2, 4, 2, 40000, 10
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, n + steps) as g:
        g.set_controller(cw)
        kq.kvq_set_splits(g.ctx, splits)
        K, V = _kv(rng, B, n, H)
        bits = BITS[rng.choice(4, size=(B, n))]
        oc.append(K, V, bits)
        g.append(0, K, V, bits)
        launches = _run_steps(gu, oracle, g, oc, cw, rng, B, Hq, H, steps, "step on a long cache, splits=%d" % splits, first_pos=n)
        assert launches == steps
        gu.assert_store_equals_oracle(g, 0, oc, pos0=n - 64, n=64 + steps)


@pytest.mark.parametrize("hidden,seed", [(128, 2), (100, 9), (7, 5), (1, 4)])
@pytest.mark.parametrize("n", [150, 40000])
def test_steps_with_controllers_of_other_widths_take_one_launch_each(gu, oracle, hidden, seed, n):
    """The paper's hidden width (128) and ragged ones, on a short cache (16-warp CTAs) and on a long one (four-warp
    CTAs): the storing CTAs of the launch evaluate the controller and publish the class, the attending warps pick it
    up; decisions bit for bit the oracle's.  A controller set later takes over."""
    rng = np.random.default_rng(hidden + n)
    cw = synth.controller_weights(seed, hidden)
    B, Hq, H, steps = 3, 6, 2, 12 if n > 1000 else 40
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, n + steps + 5) as g:
        g.set_controller(cw)
        K, V = _kv(rng, B, n, H)
        bits = BITS[rng.choice(4, size=(B, n))]
        oc.append(K, V, bits)
        g.append(0, K, V, bits)
        launches = _run_steps(gu, oracle, g, oc, cw, rng, B, Hq, H, steps, "step with hidden width %d, n=%d" % (hidden, n),
                              feat_seed=seed, first_pos=n)
        assert launches == steps
        cw2 = synth.controller_weights(322, 32)
        g.set_controller(cw2)
        _run_steps(gu, oracle, g, oc, cw2, rng, B, Hq, H, 5, "step after a change of controller", first_pos=n + steps)
        gu.assert_store_equals_oracle(g, 0, oc, pos0=max(0, n - 64), n=min(n, 64) + steps + 5)


@pytest.mark.parametrize("case", ["hidden 128", "two scale groups", "per-channel keys"])
def test_steps_of_the_other_layouts_and_controller_widths(gu, oracle, case):
    """Two scale groups per row and a wider controller (20 KV heads: two storing CTAs per sequence) take the
    one-launch kernel too; per-channel keys run the two kernels behind the same call.  Same results either way."""
    rng = np.random.default_rng(len(case))
    hidden = 128 if case == "hidden 128" else 32
    cw = synth.controller_weights(2 if hidden == 128 else 322, hidden)
    B, Hq, H, steps = 2, 4, 2, 20
    if case == "hidden 128":
        Hq = H = 20
    n = 300
    if case == "two scale groups":
        oc = oracle.GroupedOracleCache(B, Hq, H, 2)
        g = gu.GpuCache(1, B, Hq, H, n + steps, scale_groups=2)
    elif case == "per-channel keys":
        oc = oracle.PerChannelKCache(B, Hq, H)
        g = gu.GpuCache(1, B, Hq, H, n + steps, k_per_channel=True)
    else:
        oc = oracle.OracleCache(B, Hq, H)
        g = gu.GpuCache(1, B, Hq, H, n + steps)
    with g:
        g.set_controller(cw)
        K, V = _kv(rng, B, n, H)
        bits = BITS[rng.choice(4, size=(B, n))]
        oc.append(K, V, bits)
        g.append(0, K, V, bits)
        launches = _run_steps(gu, oracle, g, oc, cw, rng, B, Hq, H, steps, "step, %s" % case, first_pos=n)
        assert launches >= 2 * steps if case == "per-channel keys" else launches == steps
        if case != "per-channel keys":
            gu.assert_store_equals_oracle(g, 0, oc)


@pytest.mark.parametrize("bits", [2, 4, 8, 16])
def test_steps_with_degenerate_rows(gu, oracle, bits):
    """Rows whose quantizer takes a special path (all zero, constant, +0 and -0 mixed, a range so small that the fp16
    scale is subnormal or rounds to zero, values near the fp16 limit, one outlier channel), every token in the class
    that a bias-only controller picks: the attending warps quantize the step's token themselves, so their copy of the
    row quantizer must agree with the store's on these too."""
    rng = np.random.default_rng(bits)
    Hd = 32
    z = np.zeros
    b3 = np.zeros(4, np.float32)
    b3[[2, 4, 8, 16].index(bits)] = 1.0
    cw = synth.ControllerWeights(Hd, z((Hd, 4), np.float32), z(Hd, np.float32), z((Hd, Hd), np.float32),
                                 z(Hd, np.float32), z((4, Hd), np.float32), b3)
    B, Hq, H = 2, 4, 2
    rows = [np.zeros(64), np.full(64, 0.3125), np.where(np.arange(64) % 2 == 0, 0.0, -0.0),
            1e-4 + 1e-7 * np.arange(64), 3e-7 * (np.arange(64) % 3), np.where(np.arange(64) % 2 == 0, 60000.0, -60000.0),
            np.where(np.arange(64) == 17, 40.0, 0.01 * rng.standard_normal(64)), rng.standard_normal(64)]
    steps = len(rows)
    n = 40
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, n + steps) as g:
        g.set_controller(cw)
        K, V = _kv(rng, B, n, H)
        pre = np.full((B, n), bits, np.uint8)
        oc.append(K, V, pre)
        g.append(0, K, V, pre)
        feats = synth.features_batch(1, B, n, steps)
        for s, row in enumerate(rows):
            K1 = np.broadcast_to(row.astype(np.float16), (B, 1, H, 64)).copy()
            V1 = np.broadcast_to(rows[(s + 3) % steps].astype(np.float16), (B, 1, H, 64)).copy()
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            oc.append(K1, V1, np.full((B, 1), bits, np.uint8))
            got, out = _step(gu, g, 0, feats[:, s], K1, V1, Q)
            assert np.all(got == bits)
            gu.assert_attention_close(out, oc.decode_attn(Q), "degenerate rows, %d bits, step %d" % (bits, s))
        gu.assert_store_equals_oracle(g, 0, oc)


def test_steps_on_a_layer_of_ragged_lengths(gu, oracle):
    """Sequences of different lengths (one of them empty before the first step): every sequence against its own
    oracle cache."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(77)
    cw = synth.controller_weights(322, 32)
    B, Hq, H, steps = 3, 6, 2, 9
    lens = [200, 0, 57]
    ocs = [oracle.OracleCache(1, Hq, H) for _ in range(B)]
    with gu.GpuCache(1, B, Hq, H, 200 + steps) as g:
        g.set_controller(cw)
        K, V = _kv(rng, B, 200, H)
        bits = BITS[rng.choice(4, size=(B, 200))]
        kq.kvq_append_ragged(g.ctx, 0, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits), None, 200, lens)
        for b in range(B):
            if lens[b]:
                ocs[b].append(K[b:b + 1, :lens[b]], V[b:b + 1, :lens[b]], bits[b:b + 1, :lens[b]])
        feats = synth.features_batch(11, B, 0, steps)
        want_bits, want_logits, gap = oracle.select_bits(feats, 32, *cw.as_tuple())
        got_bits = np.zeros_like(want_bits)
        launches0 = kq.kvq_launch_count(g.ctx)
        for s in range(steps):
            K, V = _kv(rng, B, 1, H)
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            got_bits[:, s], out = _step(gu, g, 0, feats[:, s], K, V, Q)
            for b in range(B):
                ocs[b].append(K[b:b + 1], V[b:b + 1], want_bits[b:b + 1, s:s + 1])
                gu.assert_attention_close(out[b:b + 1], ocs[b].decode_attn(Q[b:b + 1]), "ragged step %d seq %d" % (s, b))
        near = gu.compare_decisions(got_bits, want_bits, want_logits, gap, "steps on ragged lengths")
        assert all(r[3] == r[4] for r in near)
        assert kq.kvq_launch_count(g.ctx) - launches0 == steps
        for b in range(B):
            for pos in sorted({0, lens[b] // 2, lens[b], lens[b] + steps - 1}):
                bt, ps, kc, vc, km, vm = kq.kvq_export_token(g.ctx, 0, b, pos, H)
                assert bt == int(ocs[b].bits[0, pos]) and ps == int(ocs[b].pool_slot[0, pos]), (b, pos)
                assert np.array_equal(kc, ocs[b].kc[0, pos]) and np.array_equal(vc, ocs[b].vc[0, pos]), (b, pos)
                assert np.array_equal(km, ocs[b].km[0, pos]) and np.array_equal(vm, ocs[b].vm[0, pos]), (b, pos)
        assert kq.kvq_seq_lens(g.ctx, 0, B).tolist() == [l + steps for l in lens]
        assert kq.kvq_device_status(g.ctx) == 0


def test_step_argument_and_capacity_errors(gu):
    import torch
    from paper_2604_04722_b200 import binding as kq
    B, Hq, H = 1, 2, 1
    with gu.GpuCache(1, B, Hq, H, 2) as g:
        f = torch.zeros((B, 4), device=gu.DEV)
        K = torch.zeros((B, 1, H, 64), dtype=torch.float16, device=gu.DEV)
        Q = torch.zeros((B, Hq, 64), dtype=torch.float16, device=gu.DEV)
        O = torch.zeros_like(Q)
        with pytest.raises(kq.KvqError) as e:
            kq.kvq_decode_step(g.ctx, 0, f, K, K, Q, O)
        assert e.value.code == kq.KVQ_ERR_NO_CONTROLLER
        g.set_controller(synth.controller_weights(322, 32))
        with pytest.raises(kq.KvqError) as e:
            kq.kvq_decode_step(g.ctx, 3, f, K, K, Q, O)
        assert e.value.code == kq.KVQ_ERR_ARG
        kq.kvq_decode_step(g.ctx, 0, f, K, K, Q, O)
        kq.kvq_decode_step(g.ctx, 0, f, K, K, Q, O)
        with pytest.raises(kq.KvqError) as e:
            kq.kvq_decode_step(g.ctx, 0, f, K, K, Q, O)
        assert e.value.code == kq.KVQ_ERR_CAPACITY
        torch.cuda.synchronize()
        assert kq.kvq_device_status(g.ctx) == 0
