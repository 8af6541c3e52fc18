"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded
inputs.  Decisions, slots, packed codes and scale/zero-point bit-exact; attention within
2e-3 + 1e-2*|ref| (fp16 output, fp32 accumulation)."""
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


# ------------------------------------------------------------------ controller

@pytest.mark.parametrize("hidden,seed,n", [(32, 322, 5000), (32, 98, 1), (128, 2, 777), (7, 5, 130)])
def test_select_bits_bit_exact(gu, oracle, hidden, seed, n):
    cw = synth.controller_weights(seed, hidden)
    feats = synth.features(seed, 0, 0, n)
    want_bits, want_logits, gap = oracle.select_bits(feats, hidden, *cw.as_tuple())
    with gu.GpuCache(1, 1, 1, 1, 32) as g:
        g.set_controller(cw)
        bits, logits = g.select_bits(feats)
    assert np.array_equal(logits.view(np.uint32), want_logits.view(np.uint32))
    # near ties (top-two gap < 1e-5) are listed in the run's summary; everything else must agree exactly
    gu.compare_decisions(bits, want_bits, want_logits, gap, "select_bits H=%d seed=%d n=%d" % (hidden, seed, n))


def test_select_bits_special_values(gu, oracle):
    """Ties, the fused-multiply-add trap and NaN features follow the oracle's rules."""
    hidden = 4
    z = lambda *s: np.zeros(s, np.float32)
    W1, b1, W2, b2, W3, b3 = z(4, 4), z(4), z(4, 4), z(4), z(4, 4), z(4)
    a = np.float32(1 + 2.0 ** -12)
    W1[0, 0] = a
    b1[0] = -np.float32(1 + 2.0 ** -11)
    W2[0, 0] = 1
    W3[1, 0] = 1
    b3[:] = [0, 0, -1, -1]
    feats = np.array([[a, 0, 0, 0], [np.nan, 1, 1, 1], [2, 0, 0, 0], [np.inf, 0, 0, 0]], np.float32)
    want_bits, want_logits, _ = oracle.select_bits(feats, hidden, W1, b1, W2, b2, W3, b3)
    cw = synth.ControllerWeights(hidden, W1, b1, W2, b2, W3, b3)
    with gu.GpuCache(1, 1, 1, 1, 32) as g:
        g.set_controller(cw)
        bits, logits = g.select_bits(feats)
    assert np.array_equal(bits, want_bits) and bits[0] == 2 and bits[2] == 4
    nan = np.isnan(want_logits)                 # NaN payload bits are not part of the contract
    assert np.array_equal(np.isnan(logits), nan)
    assert np.array_equal(logits[~nan].view(np.uint32), want_logits[~nan].view(np.uint32))


# ------------------------------------------------------------------ quantize-append

def _kv(rng, B, n, H, scale=1.0):
    K = (rng.standard_normal((B, n, H, 64)) * scale).astype(np.float16)
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    return K, V


@pytest.mark.parametrize("bt", [2, 4, 8, 16])
@pytest.mark.parametrize("n", [1, 33, 300])
def test_append_uniform_precision_bit_exact(gu, oracle, bt, n):
    rng = np.random.default_rng(bt * 1000 + n)
    B, Hq, H = 2, 4, 2
    K, V = _kv(rng, B, n, H, 3.0)
    bits = np.full((B, n), bt, np.uint8)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, bits)
    with gu.GpuCache(1, B, Hq, H, n + 5) as g:
        g.append(0, K, V, bits)
        gu.assert_store_equals_oracle(g, 0, oc)


def test_append_mixed_multi_chunk_and_incremental(gu, oracle):
    """A ragged multi-chunk prefill (3 chunks of 256), then single-token steps, then a 40-token
    append: slots continue across calls and every row is bit-exact."""
    rng = np.random.default_rng(11)
    B, Hq, H = 3, 9, 3
    sizes = [700, 1, 1, 1, 40, 257]
    total = sum(sizes)
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(2, B, Hq, H, total) as g:
        for n in sizes:
            K, V = _kv(rng, B, n, H, 2.0)
            bits = BITS[rng.choice(4, size=(B, n), p=[.4, .35, .2, .05])]
            oc.append(K, V, bits)
            g.append(1, K, V, bits)                 # layer 1; layer 0 stays empty
        gu.assert_store_equals_oracle(g, 1, oc)
        counts, resident, ebits = __import__("paper_2604_04722_b200.binding", fromlist=["x"]).kvq_stats(g.ctx, 1, B)
        assert np.array_equal(counts, oc.counts)
        rowbytes = {2: 40, 4: 72, 8: 136, 16: 256}
        assert resident == sum(rowbytes[int(b)] for b in oc.bits.ravel()) * H
        assert abs(ebits - oc.bits.astype(np.float64).mean()) < 1e-9      # E[b] = sum p(b) b, Eq. 11


def test_append_degenerate_rows_bit_exact(gu, oracle):
    """Constant rows, zeros of both signs, the fp16 maximum, subnormal ranges, huge ranges."""
    rows = []
    rows.append(np.full(64, 1.5))
    rows.append(np.zeros(64))
    r = np.zeros(64); r[::2] = -0.0; rows.append(r)
    r = np.zeros(64); r[0] = 65504; r[1] = -65504; rows.append(r)
    r = np.arange(64) * 2.0 ** -24; rows.append(r)                  # subnormal inputs and scale
    r = np.zeros(64); r[:6] = np.arange(6) * 2.0 ** -24; rows.append(r)
    r = np.linspace(-3, 3, 64); rows.append(r)
    r = np.full(64, -7.25); r[63] = -7.2421875; rows.append(r)      # range of one fp16 ulp
    x = np.stack(rows).astype(np.float16)                            # [n][64]
    n = x.shape[0]
    K = np.repeat(x[None, :, None, :], 2, axis=2).copy()             # B=1, H=2
    K[:, :, 1] = K[:, ::-1, 0]
    V = K[:, ::-1].copy()
    oc_all, B, Hq, H = [], 1, 2, 2
    for bt in (2, 4, 8, 16):
        bits = np.full((B, n), bt, np.uint8)
        oc = oracle.OracleCache(B, Hq, H)
        oc.append(K, V, bits)
        with gu.GpuCache(1, B, Hq, H, n) as g:
            g.append(0, K, V, bits)
            gu.assert_store_equals_oracle(g, 0, oc)
            Q = np.random.default_rng(bt).standard_normal((B, Hq, 64)).astype(np.float16)
            out = g.decode(0, Q)
            assert np.all(np.isfinite(out.view(np.float16)))
            gu.assert_attention_close(out, oc.decode_attn(Q), "degenerate b=%d" % bt)


def test_fused_append_equals_select_then_append(gu, oracle):
    wl = synth.CONFIGS["cfg2"]
    cw = synth.controller_weights(wl.mlp_seed, 32)
    rng = np.random.default_rng(21)
    B, Hq, H = 2, 6, 2
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, 1200) as g:
        g.set_controller(cw)
        for t0, n in ((0, 900), (900, 1), (901, 1), (902, 200)):     # multi-chunk, decode steps, one chunk
            K, V = _kv(rng, B, n, H)
            feats = synth.features_batch(5, B, t0, n)
            want_bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
            got_bits = g.append_fused(0, K, V, feats)
            assert np.array_equal(got_bits, want_bits)
            oc.append(K, V, want_bits)
        assert len(set(oc.bits.ravel().tolist())) >= 3               # the controller really mixes classes
        gu.assert_store_equals_oracle(g, 0, oc)


def test_bad_bit_width_is_flagged_not_faulted(gu, oracle):
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(1)
    K, V = _kv(rng, 1, 4, 1)
    bits = np.array([[2, 3, 8, 16]], np.uint8)
    with gu.GpuCache(1, 1, 1, 1, 8) as g:
        g.append(0, K, V, bits)
        assert kq.kvq_device_status(g.ctx) & 1
        assert kq.kvq_device_status(g.ctx) == 0                      # cleared on read
        b, *_ = g.export(0, 0, 4)
        assert b.tolist() == [[2, 16, 8, 16]]                        # the bad one is kept as fp16


def test_capacity_empty_and_argument_errors(gu):
    from paper_2604_04722_b200 import binding as kq
    import torch
    rng = np.random.default_rng(2)
    with gu.GpuCache(1, 1, 2, 1, 6) as g:
        Q = gu.dev(rng.standard_normal((1, 2, 64)).astype(np.float16).view(np.uint16))
        O = torch.zeros_like(Q)
        assert kq.lib().kvq_decode_attn(g.ctx, 0, Q.data_ptr(), O.data_ptr(), None) == kq.KVQ_ERR_EMPTY
        K, V = _kv(rng, 1, 6, 1)
        g.append(0, K, V, np.full((1, 6), 4, np.uint8))              # exactly to max_ctx
        Kd, Vd, bd = gu.dev(K[:, :1].view(np.uint16)), gu.dev(V[:, :1].view(np.uint16)), gu.dev(np.full((1, 1), 4, np.uint8))
        assert kq.lib().kvq_append(g.ctx, 0, Kd.data_ptr(), Vd.data_ptr(), bd.data_ptr(), 1, None) == kq.KVQ_ERR_CAPACITY
        assert kq.kvq_seq_len(g.ctx, 0) == 6
        assert kq.lib().kvq_append(g.ctx, 3, Kd.data_ptr(), Vd.data_ptr(), bd.data_ptr(), 1, None) == kq.KVQ_ERR_ARG
        assert kq.lib().kvq_append(g.ctx, 0, Kd.data_ptr() + 2, Vd.data_ptr(), bd.data_ptr(), 1, None) == kq.KVQ_ERR_ARG
        f = gu.dev(np.zeros((1, 1, 4), np.float32))
        assert kq.lib().kvq_append_fused(g.ctx, 0, Kd.data_ptr(), Vd.data_ptr(), f.data_ptr(), 1, None, None) == kq.KVQ_ERR_NO_CONTROLLER
        kq.kvq_reset(g.ctx)
        assert kq.kvq_seq_len(g.ctx, 0) == 0
        g.append(0, K[:, :2], V[:, :2], np.full((1, 2), 2, np.uint8))   # usable again after reset
        assert kq.kvq_stats(g.ctx, 0, 1)[0].tolist() == [[2, 0, 0, 0]]


# ------------------------------------------------------------------ decode attention

def _attend_case(gu, oracle, rng, B, Hq, H, n, bits, splits=(0,), kscale=1.5):
    K, V = _kv(rng, B, n, H, kscale)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, bits)
    want = oc.decode_attn(Q)
    from paper_2604_04722_b200 import binding as kq
    with gu.GpuCache(1, B, Hq, H, n) as g:
        g.append(0, K, V, bits)
        for s in splits:
            kq.kvq_set_splits(g.ctx, s)
            gu.assert_attention_close(g.decode(0, Q), want, "n=%d splits=%d" % (n, s))


@pytest.mark.parametrize("n", [1, 8, 31, 32, 33, 257, 1500])
def test_decode_mixed_precision_sizes(gu, oracle, n):
    rng = np.random.default_rng(n)
    B, Hq, H = 2, 6, 2
    bits = BITS[rng.choice(4, size=(B, n), p=[.4, .35, .2, .05])]
    _attend_case(gu, oracle, rng, B, Hq, H, n, bits, splits=(0, 1, 2, 7, 64))


@pytest.mark.parametrize("bt", [2, 4, 8, 16])
def test_decode_single_pool_and_empty_pools(gu, oracle, bt):
    """All tokens in one pool (the static uniform-precision baselines): three pools are empty."""
    rng = np.random.default_rng(100 + bt)
    B, Hq, H, n = 1, 4, 4, 700
    _attend_case(gu, oracle, rng, B, Hq, H, n, np.full((B, n), bt, np.uint8), splits=(0, 3))


def test_decode_all_fp16_matches_exact_softmax_attention(gu, oracle):
    """The all-fp16 cache is plain softmax attention; compare with a library routine in fp64."""
    import torch
    rng = np.random.default_rng(9)
    B, Hq, H, n = 2, 6, 3, 900
    K, V = _kv(rng, B, n, H)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    with gu.GpuCache(1, B, Hq, H, n) as g:
        g.append(0, K, V, np.full((B, n), 16, np.uint8))
        out = g.decode(0, Q)
    q = torch.from_numpy(Q.astype(np.float64)).unsqueeze(2)
    k = torch.from_numpy(K.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(2, 1)
    v = torch.from_numpy(V.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(2, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v).squeeze(2).numpy()
    gu.assert_attention_close(out, ref.astype(np.float16).view(np.uint16), "all-fp16")


def test_decode_peaked_softmax_and_large_logits(gu, oracle):
    """One dominant key (weight ~1 on one token) and keys scaled so logits span hundreds."""
    rng = np.random.default_rng(13)
    B, Hq, H, n = 1, 2, 2, 400
    bits = BITS[rng.choice(4, size=(B, n))]
    _attend_case(gu, oracle, rng, B, Hq, H, n, bits, splits=(0, 5), kscale=12.0)


@pytest.mark.parametrize("qscale,spread", [(1.0, 8.0), (0.01, 8.0), (30.0, 1.0), (1.0, 64.0), (1.0, 1000.0)])
def test_decode_query_dynamic_range(gu, oracle, qscale, spread):
    """The K-side dot product runs on a fixed-point copy of the query row: rows with outlier
    channels (some elements `spread` times larger than the rest), very small and very large rows must
    stay inside the attention tolerance.  The quantized keys carry x8 outlier channels as well."""
    rng = np.random.default_rng(int(qscale * 100 + spread))
    B, Hq, H, n = 2, 6, 2, 1100
    bits = BITS[rng.choice(4, size=(B, n), p=[.4, .35, .2, .05])]
    K, V = _kv(rng, B, n, H)
    K[:, :, :, [3, 17, 40, 55]] *= np.float16(8.0)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float32) * qscale
    Q[:, :, [5, 17, 33, 60]] *= spread
    Q = Q.astype(np.float16)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, bits)
    with gu.GpuCache(1, B, Hq, H, n) as g:
        g.append(0, K, V, bits)
        gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "qscale=%g spread=%g" % (qscale, spread))


def test_decode_after_incremental_steps(gu, oracle):
    """Prefill, then decode steps that append one token and attend (Eq. 4 then Eq. 5 each step)."""
    rng = np.random.default_rng(17)
    B, Hq, H = 2, 9, 3
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, 300) as g:
        K, V = _kv(rng, B, 250, H)
        bits = BITS[rng.choice(4, size=(B, 250))]
        oc.append(K, V, bits)
        g.append(0, K, V, bits)
        for step in range(12):
            K, V = _kv(rng, B, 1, H)
            bits = BITS[rng.choice(4, size=(B, 1))]
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            oc.append(K, V, bits)
            g.append(0, K, V, bits)
            gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "step %d" % step)


@pytest.mark.parametrize("hidden,seed", [(32, 322), (128, 2), (7, 5), (100, 9)])
def test_decode_steps_with_the_controller_inside_the_append(gu, oracle, hidden, seed):
    """Decode steps through kvq_append_fused with one new token per sequence: the one-launch token append takes the
    decision itself for every hidden width (the paper's 128 included), bit for bit the oracle's; store and attention
    follow.  20 KV heads: two warps per sequence take the same decision."""
    rng = np.random.default_rng(hidden)
    cw = synth.controller_weights(seed, hidden)
    B, Hq, H, steps = 3, 20, 20, 40
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, 64) as g:
        g.set_controller(cw)
        feats = synth.features_batch(seed, B, 0, steps)
        want_bits, want_logits, gap = oracle.select_bits(feats, hidden, *cw.as_tuple())
        got_bits = np.zeros_like(want_bits)
        for step in range(steps):
            K, V = _kv(rng, B, 1, H)
            got_bits[:, step:step + 1] = g.append_fused(0, K, V, feats[:, step:step + 1])
            oc.append(K, V, want_bits[:, step:step + 1])
        near = gu.compare_decisions(got_bits, want_bits, want_logits, gap, "token append H=%d" % hidden)
        assert all(r[3] == r[4] for r in near)
        assert len(set(want_bits.ravel().tolist())) >= 2          # the weights do spread the tokens over classes
        gu.assert_store_equals_oracle(g, 0, oc)
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "H=%d" % hidden)


@pytest.mark.parametrize("buffers", ["pageable", "page-locked", "page-locked but one", "page-locked, misaligned"])
def test_decode_step_host_matches_device_path(gu, oracle, buffers):
    """The host-buffer entry point (fused append + attention, the step's inputs and result crossing the bus)
    against the oracle: with pageable buffers it copies through staging; with page-locked ones the kernels
    reach them directly; one pageable buffer or a misaligned one sends the call back through staging."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    cw = synth.controller_weights(322, 32)
    rng = np.random.default_rng(19)
    B, Hq, H = 2, 6, 2
    oc = oracle.OracleCache(B, Hq, H)

    def host(a, keep_pageable=False):
        """numpy array a as the kind of host buffer under test (returns the object to pass and a numpy view)."""
        a = np.ascontiguousarray(a)
        raw = a.view(np.uint8).reshape(-1)
        if buffers == "pageable" or keep_pageable:
            return a, a
        pad = 8 if buffers == "page-locked, misaligned" else 0
        t = torch.zeros(raw.size + pad, dtype=torch.uint8).pin_memory()
        t[pad:] = torch.from_numpy(raw.copy())
        view = t[pad:].numpy().view(a.dtype).reshape(a.shape)
        return t.data_ptr() + pad, view

    with gu.GpuCache(1, B, Hq, H, 80) as g:
        g.set_controller(cw)
        K, V = _kv(rng, B, 64, H)
        feats = synth.features_batch(1, B, 0, 64)
        bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
        oc.append(K, V, bits)
        assert np.array_equal(g.append_fused(0, K, V, feats), bits)
        for step in range(4):
            K, V = _kv(rng, B, 1, H)
            feats = synth.features_batch(1, B, 64 + step, 1)
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            f_h, _ = host(feats[:, 0].astype(np.float32))
            k_h, _ = host(K)
            v_h, _ = host(V, keep_pageable=(buffers == "page-locked but one"))
            q_h, _ = host(Q)
            o_h, O = host(np.zeros((B, Hq, 64), np.uint16))
            got_bits = np.zeros(B, np.uint8)
            kq.kvq_decode_step_host(g.ctx, 0, f_h, k_h, v_h, q_h, o_h, got_bits)
            want_bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
            assert np.array_equal(got_bits, want_bits[:, 0])
            oc.append(K, V, want_bits)
            gu.assert_attention_close(O, oc.decode_attn(Q), "host step %d (%s)" % (step, buffers))
        gu.assert_store_equals_oracle(g, 0, oc)


# ------------------------------------------------------------------ several causal query rows

@pytest.mark.parametrize("T,n", [(1, 200), (4, 333), (8, 1500), (11, 90), (20, 700)])
def test_attend_last_is_causal_attention_at_each_of_the_last_positions(gu, oracle, T, n):
    """kvq_attend_last: query row i sits at position n - T + i and sees positions <= its own (Eq. 5 applied
    at each of the last T positions).  The oracle computes every row on a cache truncated after its
    position; rows 8 and up go through a second launch."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(1000 * T + n)
    B, Hq, H = 2, 6, 2
    bits = BITS[rng.choice(4, size=(B, n), p=[.4, .3, .2, .1])]
    K, V = _kv(rng, B, n, H)
    Q = rng.standard_normal((B, T, Hq, 64)).astype(np.float16)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, bits)
    want = oc.attend_last(Q)
    with gu.GpuCache(1, B, Hq, H, n) as g:
        g.append(0, K[:, :n - T], V[:, :n - T], bits[:, :n - T])       # the cache, then the T new tokens at once
        g.append(0, K[:, n - T:], V[:, n - T:], bits[:, n - T:])
        Qd = gu.dev(Q.view(np.uint16))
        for splits in (0, 3):
            kq.kvq_set_splits(g.ctx, splits)
            O = torch.zeros_like(Qd)
            kq.kvq_attend_last(g.ctx, 0, Qd, O, T)
            torch.cuda.synchronize()
            gu.assert_attention_close(O.cpu().numpy().view(np.uint16), want, "T=%d n=%d splits=%d" % (T, n, splits))
        # the last row is the ordinary decode step
        gu.assert_attention_close(g.decode(0, np.ascontiguousarray(Q[:, T - 1])), want[:, T - 1], "last row")
        assert kq.lib().kvq_attend_last(g.ctx, 0, Qd.data_ptr(), O.data_ptr(), n + 1, None) == kq.KVQ_ERR_ARG


# ------------------------------------------------------------------ determinism

def test_two_runs_give_the_same_bits(gu):
    """The same appends and the same query twice, on two handles: packed rows, scales and the attention output
    are bitwise equal (slots come from a scan, not from atomics; partial results are merged in record order
    whichever warp arrives last)."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(123)
    B, Hq, H, n = 2, 8, 4, 3000
    K, V = _kv(rng, B, n, H)
    bits = BITS[rng.choice(4, size=(B, n), p=[.4, .3, .2, .1])]
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    runs = []
    for _ in range(2):
        with gu.GpuCache(1, B, Hq, H, n) as g:
            g.append(0, K[:, :2000], V[:, :2000], bits[:, :2000])
            g.append(0, K[:, 2000:], V[:, 2000:], bits[:, 2000:])
            outs = []
            for splits in (0, 7):
                kq.kvq_set_splits(g.ctx, splits)
                outs += [g.decode(0, Q), g.decode(0, Q)]
            runs.append((g.export(0, 0, n), outs))
    for a, b in zip(runs[0][0], runs[1][0]):
        assert np.array_equal(a, b)
    for a, b in zip(runs[0][1], runs[1][1]):
        assert np.array_equal(a, b)
    assert np.array_equal(runs[0][1][0], runs[0][1][1]) and np.array_equal(runs[0][1][2], runs[0][1][3])


@pytest.mark.parametrize("seed", range(12))
def test_decode_with_extreme_value_scales_peaks_and_query_ranges(gu, oracle, seed):
    """The value weights p * scale_v go through an integer grid shared by many tiles and the query through a
    fixed-point grid: value rows whose scales differ by up to 2^22 from token to token, a single dominant key over a
    flat background, query channels of very different size and very small or large queries must all stay within the
    attention tolerance, for the automatic plan and for an explicit split count, in two appends."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(1000 + seed)
    B, H = int(rng.choice([1, 2])), int(rng.choice([1, 3]))
    Hq = H * int(rng.choice([1, 3]))
    n = [5, 40, 333, 1500, 5000, 777][seed % 6]
    mix = rng.dirichlet(np.ones(4) * 0.7)
    kscale = [0.05, 1.0, 4.0, 12.0][seed % 4]
    K = (rng.standard_normal((B, n, H, 64)) * kscale).astype(np.float16)
    vs = np.exp2(rng.integers(-12, 11, size=(B, n, H, 1))).astype(np.float32)
    V = np.clip(rng.standard_normal((B, n, H, 64)) * vs, -60000, 60000).astype(np.float16)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float32)
    mode = seed % 4
    if mode == 1:                                            # one dominant key
        for b in range(B):
            for h in range(Hq):
                K[b, int(rng.integers(0, n)), h // (Hq // H)] = (Q[b, h] * 4.0).astype(np.float16)
    if mode == 2:
        Q *= np.exp2(rng.integers(-8, 8, size=(B, Hq, 64)))
    if mode == 3:
        Q *= [1e-3, 30.0][seed % 2]
    Q = Q.astype(np.float16)
    bits = BITS[rng.choice(4, size=(B, n), p=mix)]
    oc = oracle.OracleCache(B, Hq, H)
    with gu.GpuCache(1, B, Hq, H, n) as g:
        cut = int(rng.integers(1, n + 1))
        for lo, hi in ((0, cut), (cut, n)):
            if hi > lo:
                g.append(0, K[:, lo:hi], V[:, lo:hi], bits[:, lo:hi])
                oc.append(K[:, lo:hi], V[:, lo:hi], bits[:, lo:hi])
        want = oc.decode_attn(Q)
        for splits in (0, [1, 2, 5, 16, 64][seed % 5]):
            kq.kvq_set_splits(g.ctx, splits)
            gu.assert_attention_close(g.decode(0, Q), want, "seed %d splits %d" % (seed, splits))
        assert kq.kvq_device_status(g.ctx) == 0
