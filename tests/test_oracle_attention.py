"""Pins for the oracle's decode attention (Eq. 5 over the mixed-precision cache) -- CPU only."""
import math

import numpy as np
import torch

from paper_2604_04722_b200 import synth

BITS = np.array([2, 4, 8, 16], np.uint8)


def _f16(u16):
    return np.asarray(u16, np.uint16).view(np.float16).astype(np.float64)


def _make(oracle, rng, B, Hq, Hkv, n, bits):
    K = (rng.standard_normal((B, n, Hkv, 64)) * 1.5).astype(np.float16)
    V = rng.standard_normal((B, n, Hkv, 64)).astype(np.float16)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    cache = oracle.OracleCache(B, Hq, Hkv)
    cache.append(K, V, bits)
    return K, V, Q, cache


def test_all_fp16_cache_equals_library_softmax_attention(oracle):
    """With every token at 16 bits the cache holds K and V unchanged, so the result must be the
    fp64 scaled-dot-product attention of a library routine, grouped heads included."""
    rng = np.random.default_rng(0)
    B, Hq, Hkv, n = 2, 6, 2, 193
    bits = np.full((B, n), 16, np.uint8)
    K, V, Q, cache = _make(oracle, rng, B, Hq, Hkv, n, bits)
    out, out64 = cache.decode_attn(Q, want64=True)
    g = Hq // Hkv
    q = torch.from_numpy(Q.astype(np.float64)).unsqueeze(2)                       # [B][Hq][1][D]
    k = torch.from_numpy(K.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(g, 1)
    v = torch.from_numpy(V.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(g, 1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v).squeeze(2).numpy()
    assert np.allclose(out64, ref, rtol=1e-12, atol=1e-13)
    assert np.array_equal(out, ref.astype(np.float16).view(np.uint16))


def test_brute_force_on_eight_token_caches(oracle):
    """Eq. 5 written out term by term in Python floats over the dequantized rows."""
    rng = np.random.default_rng(1)
    B, Hq, Hkv, n = 2, 4, 2, 8
    bits = BITS[rng.integers(0, 4, size=(B, n))]
    bits[0, :4] = [2, 4, 8, 16]
    K, V, Q, cache = _make(oracle, rng, B, Hq, Hkv, n, bits)
    _, out64 = cache.decode_attn(Q, want64=True)
    for b in range(B):
        for h in range(Hq):
            kvh = h // (Hq // Hkv)
            q = [float(x) for x in Q[b, h]]
            z, vrows = [], []
            for t in range(n):
                bt = int(bits[b, t])
                khat = oracle.dequantize_row(cache.kc[b, t, kvh, :64 * bt // 8], cache.km[b, t, kvh], 64, bt)
                vhat = oracle.dequantize_row(cache.vc[b, t, kvh, :64 * bt // 8], cache.vm[b, t, kvh], 64, bt)
                z.append(math.fsum(q[i] * float(khat[i]) for i in range(64)) / 8.0)
                vrows.append([float(x) for x in vhat])
            zmax = max(z)
            e = [math.exp(x - zmax) for x in z]
            den = math.fsum(e)
            for i in range(64):
                want = math.fsum(e[t] / den * vrows[t][i] for t in range(n))
                assert abs(out64[b, h, i] - want) <= 1e-12 * max(1.0, abs(want))


def test_single_token_returns_its_value_row_and_group_mapping(oracle):
    """One cached token: softmax weight 1, so O = vhat of KV head h // g, exactly."""
    rng = np.random.default_rng(2)
    B, Hq, Hkv = 1, 9, 3
    for bt in (2, 4, 8, 16):
        bits = np.full((B, 1), bt, np.uint8)
        K, V, Q, cache = _make(oracle, rng, B, Hq, Hkv, 1, bits)
        out = cache.decode_attn(Q)
        for h in range(Hq):
            vhat = oracle.dequantize_row(cache.vc[0, 0, h // 3, :64 * bt // 8], cache.vm[0, 0, h // 3], 64, bt)
            assert np.array_equal(out[0, h], vhat.astype(np.float16).view(np.uint16))
        if bt == 16:
            assert np.array_equal(out[0, 4], V[0, 0, 1].view(np.uint16))


def test_identical_keys_give_the_mean_of_values(oracle):
    rng = np.random.default_rng(3)
    B, Hq, Hkv, n = 1, 2, 1, 33
    K = np.repeat(rng.standard_normal((B, 1, Hkv, 64)), n, axis=1).astype(np.float16)
    V = rng.standard_normal((B, n, Hkv, 64)).astype(np.float16)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    bits = np.full((B, n), 8, np.uint8)
    cache = oracle.OracleCache(B, Hq, Hkv)
    cache.append(K, V, bits)
    _, out64 = cache.decode_attn(Q, want64=True)
    vhat = np.stack([oracle.dequantize_row(cache.vc[0, t, 0, :64], cache.vm[0, t, 0], 64, 8) for t in range(n)])
    assert np.allclose(out64[0, 0], vhat.astype(np.float64).mean(0), rtol=1e-12, atol=1e-14)
    assert np.allclose(out64[0, 1], out64[0, 0], rtol=1e-12, atol=1e-14)


def test_output_lies_in_the_hull_of_the_value_rows_and_one_hot_limit(oracle):
    rng = np.random.default_rng(4)
    B, Hq, Hkv, n = 1, 3, 3, 120
    bits = BITS[rng.integers(0, 4, size=(B, n))]
    K, V, Q, cache = _make(oracle, rng, B, Hq, Hkv, n, bits)
    _, out64 = cache.decode_attn(Q, want64=True)
    for h in range(Hq):
        vhat = np.stack([oracle.dequantize_row(cache.vc[0, t, h, :64 * int(bits[0, t]) // 8],
                                               cache.vm[0, t, h], 64, int(bits[0, t])) for t in range(n)])
        assert np.all(out64[0, h] <= vhat.max(0) + 1e-9) and np.all(out64[0, h] >= vhat.min(0) - 1e-9)
    # a query aligned with one very large key puts all the weight on that token
    K2 = K.copy()
    K2[0, 17, 0] = (Q[0, 0].astype(np.float32) * 40).astype(np.float16)
    cache2 = oracle.OracleCache(B, Hq, Hkv)
    bits2 = bits.copy()
    bits2[0, 17] = 16
    cache2.append(K2, V, bits2)
    out = cache2.decode_attn(Q)
    assert np.array_equal(out[0, 0], V[0, 17, 0].view(np.uint16))


def test_softmax_is_invariant_to_token_order_and_appending_in_pieces(oracle):
    """The cache is a set of rows: permuting tokens (which is what walking the pools does) or
    appending them in several calls leaves Eq. 5 unchanged."""
    rng = np.random.default_rng(5)
    B, Hq, Hkv, n = 2, 4, 2, 77
    bits = BITS[rng.integers(0, 4, size=(B, n))]
    K, V, Q, cache = _make(oracle, rng, B, Hq, Hkv, n, bits)
    _, ref = cache.decode_attn(Q, want64=True)
    perm = rng.permutation(n)
    c2 = oracle.OracleCache(B, Hq, Hkv)
    c2.append(K[:, perm], V[:, perm], bits[:, perm])
    assert np.allclose(c2.decode_attn(Q, want64=True)[1], ref, rtol=1e-12, atol=1e-13)
    c3 = oracle.OracleCache(B, Hq, Hkv)
    for lo, hi in ((0, 30), (30, 31), (31, n)):
        c3.append(K[:, lo:hi], V[:, lo:hi], bits[:, lo:hi])
    assert np.array_equal(c3.decode_attn(Q), cache.decode_attn(Q))
    assert np.array_equal(c3.pool_slot, cache.pool_slot)


def test_quantized_cache_approaches_fp16_attention_with_more_bits(oracle):
    """Sanity of the whole chain: 8-bit attention is closer to the fp16 result than 4-bit, which
    is closer than 2-bit (the lever the paper's allocation relies on, Section 3.7)."""
    rng = np.random.default_rng(6)
    B, Hq, Hkv, n = 1, 4, 4, 256
    errs = {}
    K = rng.standard_normal((B, n, Hkv, 64)).astype(np.float16)
    V = rng.standard_normal((B, n, Hkv, 64)).astype(np.float16)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    outs = {}
    for bt in (2, 4, 8, 16):
        c = oracle.OracleCache(B, Hq, Hkv)
        c.append(K, V, np.full((B, n), bt, np.uint8))
        outs[bt] = c.decode_attn(Q, want64=True)[1]
    for bt in (2, 4, 8):
        errs[bt] = np.abs(outs[bt] - outs[16]).max()
    assert errs[8] < errs[4] < errs[2] and errs[8] < 5e-3


def test_workload_table_matches_the_backbones():
    """Layers/heads follow Table 1 (30/9, 32/15, 24/32); head_dim 64 and KV heads per config."""
    c = synth.CONFIGS
    assert (c["cfg2"].layers, c["cfg2"].q_heads, c["cfg2"].kv_heads) == (30, 9, 3)
    assert (c["cfg3"].layers, c["cfg3"].q_heads, c["cfg3"].kv_heads) == (32, 15, 5)
    assert (c["cfg4"].layers, c["cfg4"].q_heads, c["cfg4"].kv_heads) == (24, 32, 32)
    assert c["cfg5"].context == 32768 and c["cfg5"].batch == 16
    K, V = synth.kv_rows(0, 0, 0, 0, 4096, 3)
    assert K.dtype == np.float16 and K.shape == (4096, 3, 64)
    ch = synth.outlier_channels(0, 0, 3, 64, 1)
    sd = K.astype(np.float64).std(0)
    for h in range(3):
        big = np.zeros(64, bool)
        big[ch[h]] = True
        assert np.all(sd[h][big] > 6) and np.all(sd[h][~big] < 1.5)
    b = synth.bits_iid(0, 0, 0, 100000, c["cfg5"].mix)
    assert abs((b == 2).mean() - 0.5) < 0.01 and abs((b == 16).mean() - 0.05) < 0.005
    r = synth.bits_runs(0, 0, 0, 100000, c["cfg4"].mix, 16)
    changes = np.count_nonzero(np.diff(r.astype(int))) + 1
    assert 12 < 100000 / changes < 30          # mean run near 16 (equal neighbours merge)


def test_attend_last_matches_library_causal_attention_and_ignores_the_future(oracle):
    """Causal attention of the last T positions: an all-fp16 cache must equal a library routine with a
    causal mask (fp64), and a row's result must not move when later tokens change."""
    import torch
    rng = np.random.default_rng(21)
    B, Hq, H, n, T = 2, 4, 2, 60, 5
    K = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    Q = rng.standard_normal((B, T, Hq, 64)).astype(np.float16)
    oc = oracle.OracleCache(B, Hq, H)
    oc.append(K, V, np.full((B, n), 16, np.uint8))
    got = oc.attend_last(Q).view(np.float16).astype(np.float64)                    # [B][T][Hq][D]
    q = torch.from_numpy(Q.astype(np.float64)).permute(0, 2, 1, 3)                 # [B][Hq][T][D]
    k = torch.from_numpy(K.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(Hq // H, 1)
    v = torch.from_numpy(V.astype(np.float64)).permute(0, 2, 1, 3).repeat_interleave(Hq // H, 1)
    mask = torch.ones(T, n, dtype=torch.bool).tril(diagonal=n - T)                 # row i sees keys <= n - T + i
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask).permute(0, 2, 1, 3).numpy()
    assert np.max(np.abs(got - ref)) < 2e-3
    # change the last token only: rows 0 .. T-2 stay bit-identical, the last row moves
    K2, V2 = K.copy(), V.copy()
    K2[:, -1] *= np.float16(-3.0)
    V2[:, -1] += np.float16(5.0)
    oc2 = oracle.OracleCache(B, Hq, H)
    oc2.append(K2, V2, np.full((B, n), 16, np.uint8))
    got2 = oc2.attend_last(Q)
    assert np.array_equal(got2[:, :T - 1], oc.attend_last(Q)[:, :T - 1])
    assert not np.array_equal(got2[:, T - 1], oc.attend_last(Q)[:, T - 1])
    # one row is the plain decode step
    assert np.array_equal(oc.attend_last(Q[:, -1:])[:, 0], oc.decode_attn(np.ascontiguousarray(Q[:, -1])))
