"""Grouped scales (one {scale, zero-point} pair per 32 channels instead of per row): the CUDA path of a
cache made with scale_groups = 2 against the grouped oracle cache.  Bit-widths, slots, packed codes and all
four meta words per row bit-exact; attention within 2e-3 + 1e-2*|ref|."""
import numpy as np
import pytest

from paper_2604_04722_b200 import synth

pytestmark = pytest.mark.gpu

BITS = np.array([2, 4, 8, 16], np.uint8)
ROW_BYTES = {2: 48, 4: 80, 8: 144, 16: 256}


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_04722_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _kv(rng, B, n, H, scale=1.5):
    K = (rng.standard_normal((B, n, H, 64)) * scale).astype(np.float16)
    V = (rng.standard_normal((B, n, H, 64)) * scale).astype(np.float16)
    K[..., 32:] += np.float16(2.0)          # the two groups of a row see different ranges
    V[..., :32] *= np.float16(0.25)
    return K, V


def test_only_one_or_two_groups(gu):
    from paper_2604_04722_b200 import binding as kq
    for g in (0, 3, 4, -1):
        with pytest.raises(kq.KvqError):
            kq.kvq_create_grouped(1, 2, 2, 64, 64, 1, 0, g)
    h = kq.kvq_create_grouped(1, 2, 2, 64, 64, 1, 0, 1)       # 1 is the ordinary cache
    kq.kvq_destroy(h)


@pytest.mark.parametrize("bt", [2, 4, 8, 16])
@pytest.mark.parametrize("n", [1, 33, 300])
def test_append_uniform_precision_bit_exact(gu, oracle, bt, n):
    rng = np.random.default_rng(bt * 1000 + n)
    B, Hq, H = 2, 4, 2
    K, V = _kv(rng, B, n, H, 3.0)
    bits = np.full((B, n), bt, np.uint8)
    oc = oracle.GroupedOracleCache(B, Hq, H, 2)
    oc.append(K, V, bits)
    with gu.GpuCache(1, B, Hq, H, n + 5, scale_groups=2) as g:
        g.append(0, K, V, bits)
        gu.assert_store_equals_oracle(g, 0, oc)
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "uniform %d-bit" % bt)


def test_prefill_fused_append_steps_and_attention(gu, oracle):
    """A multi-chunk prefill with given bit-widths, a prefill chunk decided by the controller inside the
    launch, single-token steps on both paths, attention after every step; GQA with 3 query heads per KV head."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(77)
    B, Hq, H = 3, 9, 3
    cw = synth.controller_weights(322, 32)
    oc = oracle.GroupedOracleCache(B, Hq, H, 2)
    with gu.GpuCache(2, B, Hq, H, 1200, scale_groups=2) as g:
        g.set_controller(cw)
        K, V = _kv(rng, B, 700, H)
        bits = BITS[rng.choice(4, size=(B, 700), p=[.4, .35, .2, .05])]
        oc.append(K, V, bits)
        g.append(1, K, V, bits)
        K, V = _kv(rng, B, 300, H)
        feats = synth.features_batch(5, B, 0, 300)
        want_bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
        got_bits = g.append_fused(1, K, V, feats)
        assert np.array_equal(got_bits, want_bits)
        oc.append(K, V, want_bits)
        for step in range(6):
            K, V = _kv(rng, B, 1, H)
            if step % 2:
                feats = synth.features_batch(100 + step, B, 0, 1)
                bits, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
                assert np.array_equal(g.append_fused(1, K, V, feats), bits)
            else:
                bits = BITS[rng.choice(4, size=(B, 1))]
                g.append(1, K, V, bits)
            oc.append(K, V, bits)
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            gu.assert_attention_close(g.decode(1, Q), oc.decode_attn(Q), "step %d" % step)
        gu.assert_store_equals_oracle(g, 1, oc)
        counts, resident, _ = kq.kvq_stats(g.ctx, 1, B)
        assert np.array_equal(counts, oc.counts)
        assert resident == sum(ROW_BYTES[int(b)] for b in oc.bits.ravel()) * H
        # one token through the host-buffer export
        bt, ps, kc, vc, km, vm = kq.kvq_export_token(g.ctx, 1, 2, 701, H, 2)
        assert bt == oc.bits[2, 701] and ps == oc.pool_slot[2, 701]
        assert np.array_equal(kc, oc.kc[2, 701]) and np.array_equal(vc, oc.vc[2, 701])
        assert np.array_equal(km, oc.km[2, 701]) and np.array_equal(vm, oc.vm[2, 701])


@pytest.mark.parametrize("splits", [0, 1, 7, 64])
def test_long_context_over_several_blocks_and_every_split(gu, oracle, splits):
    """3000 tokens, mostly 2-bit: the 2-bit stream fills more than one 64 KB block (80 tiles of 16 tokens),
    and every pool ends in a ragged tile."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(5)
    B, Hq, H, n = 1, 2, 1, 3000
    K, V = _kv(rng, B, n, H)
    bits = BITS[rng.choice(4, size=(B, n), p=[.7, .15, .1, .05])]
    oc = oracle.GroupedOracleCache(B, Hq, H, 2)
    oc.append(K, V, bits)
    with gu.GpuCache(1, B, Hq, H, n, scale_groups=2) as g:
        g.append(0, K, V, bits)
        kq.kvq_set_splits(g.ctx, splits)
        for spread in (1.0, 64.0):
            Q = (rng.standard_normal((B, Hq, 64)) * spread).astype(np.float16)
            Q[..., ::7] *= np.float16(1.0 / 64)
            gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "splits %d spread %g" % (splits, spread))
        gu.assert_store_equals_oracle(g, 0, oc, 1200, 200)


def test_reset_and_reuse_leaves_no_stale_scales(gu, oracle):
    """After kvq_reset the blocks are handed out again; rows of the earlier fill must not reach the result."""
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(9)
    B, Hq, H = 2, 4, 2
    with gu.GpuCache(1, B, Hq, H, 400, scale_groups=2) as g:
        K, V = _kv(rng, B, 400, H, 100.0)
        K[:, ::3] = np.float16(60000.0)
        g.append(0, K, V, BITS[rng.choice(3, size=(B, 400))])
        kq.kvq_reset(g.ctx)
        oc = oracle.GroupedOracleCache(B, Hq, H, 2)
        for n in (37, 1, 1):
            K, V = _kv(rng, B, n, H)
            bits = BITS[rng.choice(4, size=(B, n))]
            g.append(0, K, V, bits)
            oc.append(K, V, bits)
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            gu.assert_attention_close(g.decode(0, Q), oc.decode_attn(Q), "after reset, +%d" % n)
        gu.assert_store_equals_oracle(g, 0, oc)


def test_ragged_batch_with_grouped_scales(gu, oracle):
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(13)
    B, Hq, H = 3, 4, 2
    lens = [290, 0, 77]
    ocs = [oracle.GroupedOracleCache(1, Hq, H, 2) for _ in range(B)]
    with gu.GpuCache(1, B, Hq, H, 400, scale_groups=2) as g:
        K, V = _kv(rng, B, 290, H)
        bits = BITS[rng.choice(4, size=(B, 290))]
        kq.kvq_append_ragged(g.ctx, 0, gu.dev(K.view(np.uint16)), gu.dev(V.view(np.uint16)), gu.dev(bits), None, 290, lens)
        for b in range(B):
            if lens[b]:
                ocs[b].append(K[b:b + 1, :lens[b]], V[b:b + 1, :lens[b]], bits[b:b + 1, :lens[b]])
        K, V = _kv(rng, B, 1, H)
        bits = BITS[rng.choice(4, size=(B, 1))]
        g.append(0, K, V, bits)
        for b in range(B):
            ocs[b].append(K[b:b + 1], V[b:b + 1], bits[b:b + 1])
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        out = g.decode(0, Q)
        for b in range(B):
            gu.assert_attention_close(out[b:b + 1], ocs[b].decode_attn(Q[b:b + 1]), "sequence %d" % b)


def test_the_other_attention_entry_points_on_a_grouped_cache(gu, oracle):
    """Causal rows for the last positions, the statistics variant, the fixed-scratch variant and the host-buffer
    step all run the same kernel template; with grouped scales each must agree with the grouped oracle."""
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng = np.random.default_rng(21)
    B, Hq, H, n, T = 2, 4, 2, 300, 3
    K, V = _kv(rng, B, n, H)
    bits = BITS[rng.choice(4, size=(B, n), p=[.4, .3, .2, .1])]
    Q = rng.standard_normal((B, T, Hq, 64)).astype(np.float16)
    with gu.GpuCache(1, B, Hq, H, n + 1, scale_groups=2) as g:
        g.append(0, K, V, bits)
        Qd = gu.dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        kq.kvq_attend_last(g.ctx, 0, Qd, O, T)
        torch.cuda.synchronize()
        got = O.cpu().numpy().view(np.uint16)
        for i in range(T):                              # row i sees positions <= n - T + i
            upto = n - T + i + 1
            oc = oracle.GroupedOracleCache(B, Hq, H, 2)
            oc.append(K[:, :upto], V[:, :upto], bits[:, :upto])
            gu.assert_attention_close(got[:, i], oc.decode_attn(np.ascontiguousarray(Q[:, i])), "row %d" % i)
        want = oc.decode_attn(np.ascontiguousarray(Q[:, T - 1]))            # the whole cache, last query row
        Ql = gu.dev(np.ascontiguousarray(Q[:, T - 1]).view(np.uint16))
        O1, O2 = torch.zeros_like(Ql), torch.zeros_like(Ql)
        var = torch.zeros(B, dtype=torch.float32, device=gu.DEV)
        kq.kvq_decode_attn_var(g.ctx, 0, Ql, O1, var)
        kq.kvq_decode_attn_static(g.ctx, 0, Ql, O2)
        torch.cuda.synchronize()
        gu.assert_attention_close(O1.cpu().numpy().view(np.uint16), want, "statistics variant")
        gu.assert_attention_close(O2.cpu().numpy().view(np.uint16), want, "fixed-scratch variant")
        assert np.all(np.isfinite(var.cpu().numpy())) and np.all(var.cpu().numpy() >= 0)
        # one step from host buffers: append a controller-decided token, then attend
        cw = synth.controller_weights(322, 32)
        g.set_controller(cw)
        Kn, Vn = _kv(rng, B, 1, H)
        feats = synth.features_batch(3, B, 0, 1).astype(np.float32)
        nb, _, _ = oracle.select_bits(feats, 32, *cw.as_tuple())
        Qh = np.ascontiguousarray(Q[:, 0])
        Oh = np.zeros_like(Qh)
        bo = np.zeros((B, 1), np.uint8)
        kq.kvq_decode_step_host(g.ctx, 0, feats, Kn.view(np.uint16), Vn.view(np.uint16), Qh.view(np.uint16),
                                Oh.view(np.uint16), bo)
        assert np.array_equal(bo, nb)
        oc.append(Kn, Vn, nb)
        gu.assert_attention_close(Oh.view(np.uint16), oc.decode_attn(Qh), "host-buffer step")
