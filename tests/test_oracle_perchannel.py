"""Pins of the per-channel key cache of the oracle: what the definition and the mathematics fix, checked against
routines that do not share its code path (the per-token cache on transposed data, a library attention)."""
import numpy as np
import pytest

BITS = np.array([2, 4, 8, 16], np.uint8)


def _rows(rng, B, n, H, D, scale=1.0):
    return (rng.standard_normal((B, n, H, D)) * scale).astype(np.float16)


@pytest.mark.parametrize("bt", [2, 4, 8])
def test_one_window_equals_the_per_token_quantizer_on_the_transposed_block(oracle, bt):
    """head_dim = window = 16: quantizing the 16 x 16 key block per channel is quantizing its transpose per token,
    so the codes are the transposed codes of the plain cache and the {scale, zero-point} pairs are equal."""
    rng = np.random.default_rng(bt)
    D = W = 16
    K = _rows(rng, 1, W, 1, D, 2.0)
    V = _rows(rng, 1, W, 1, D)
    bits = np.full((1, W), bt, np.uint8)
    pc = oracle.PerChannelKCache(1, 1, 1, head_dim=D, window=W)
    pc.append(K, V, bits)
    state, kc, khat, chan = pc.key_state()
    plain = oracle.OracleCache(1, 1, 1, head_dim=D)
    Kt = np.ascontiguousarray(K[0, :, 0, :].T)[None, :, None, :]            # token t of the plain cache = channel t
    plain.append(Kt, Kt, bits)
    nb = D * bt // 8
    mine = oracle._unpack_codes(kc[0, :, 0, :nb], D, bt)                    # [token][channel]
    theirs = oracle._unpack_codes(plain.kc[0, :, 0, :nb], D, bt)            # [channel][token]
    assert np.array_equal(mine, theirs.T) and np.all(state == 1)
    assert np.array_equal(chan[(0, 0, bt, 0)], plain.km[0, :, 0, :])


def test_open_windows_and_16_bit_tokens_keep_their_rows(oracle):
    """Fewer than 16 tokens of a precision: nothing is packed, keys are exact, and attention equals a library
    softmax attention over the fp16 keys and the per-token dequantized values."""
    import torch
    rng = np.random.default_rng(5)
    B, Hq, H, n = 2, 4, 2, 40
    K, V = _rows(rng, B, n, H, 64, 1.5), _rows(rng, B, n, H, 64)
    bits = np.tile(BITS, (B, n // 4))                                       # 10 tokens of each precision: all windows open
    pc = oracle.PerChannelKCache(B, Hq, H)
    pc.append(K, V, bits)
    state, kc, khat, chan = pc.key_state()
    assert not chan and np.all(state == 0)
    assert np.array_equal(khat, K.astype(np.float32))
    assert np.array_equal(kc[..., :128].reshape(B, n, H, 64, 2), K.view(np.uint8).reshape(B, n, H, 64, 2))
    plain = oracle.OracleCache(B, Hq, H)
    plain.append(K, V, bits)                                                # same values side
    vhat = np.empty((B, n, H, 64))
    for b in range(B):
        for t in range(n):
            for h in range(H):
                bt = int(bits[b, t])
                vhat[b, t, h] = oracle.dequantize_row(plain.vc[b, t, h, :64 * bt // 8], plain.vm[b, t, h], 64, bt)
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    got = pc.decode_attn(Q).view(np.float16).astype(np.float64)
    for b in range(B):
        for hq in range(Hq):
            h = hq // (Hq // H)
            want = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(Q[b, hq].astype(np.float64))[None, None], torch.from_numpy(K[b, :, h].astype(np.float64))[None],
                torch.from_numpy(vhat[b, :, h])[None])[0, 0].numpy()
            assert np.all(np.abs(got[b, hq] - want) <= 1e-3 * np.abs(want) + 1e-3)


def test_windows_fill_in_slot_order_and_bound_the_error_per_channel(oracle):
    """Mixed precisions: a token's key is packed exactly when its window (16 consecutive slots of its precision) is
    complete; every packed key element lies within half a channel scale of the fp16 value; an outlier channel does
    not spoil the other channels (which it does with one scale per token)."""
    rng = np.random.default_rng(9)
    B, H, n = 1, 1, 200
    K = _rows(rng, B, n, H, 64)
    K[..., 7] *= 16                                                         # one outlier channel
    V = _rows(rng, B, n, H, 64)
    bits = BITS[rng.choice(3, size=(B, n))]                                 # 2, 4, 8 bits
    pc = oracle.PerChannelKCache(B, 1, H)
    for lo in range(0, n, 37):                                              # in pieces: windows fill across calls
        pc.append(K[:, lo:lo + 37], V[:, lo:lo + 37], bits[:, lo:lo + 37])
    state, kc, khat, chan = pc.key_state()
    x = K.astype(np.float32)
    for bt in (2, 4, 8):
        pos = np.flatnonzero(bits[0] == bt)
        full = len(pos) // 16 * 16
        assert np.all(state[0, pos[:full], 0] == 1) and np.all(state[0, pos[full:], 0] == 0)
        assert np.array_equal(khat[0, pos[full:]], x[0, pos[full:]])
        for w in range(full // 16):
            s = oracle.half_to_float(chan[(0, 0, bt, w)][:, 0])
            err = np.abs(khat[0, pos[w * 16:(w + 1) * 16], 0] - x[0, pos[w * 16:(w + 1) * 16], 0])
            assert np.all(err <= s[None, :] * 0.5 * (1 + 2.0 ** -9) + 1e-6)
    plain = oracle.OracleCache(B, 1, H)
    plain.append(K, V, bits)
    pos2 = np.flatnonzero(bits[0] == 2)[:16]
    per_token = np.stack([oracle.dequantize_row(plain.kc[0, t, 0, :16], plain.km[0, t, 0], 64, 2) for t in pos2])
    others = [i for i in range(64) if i != 7]
    assert np.abs(khat[0, pos2, 0][:, others] - x[0, pos2, 0][:, others]).mean() < \
        0.5 * np.abs(per_token[:, others] - x[0, pos2, 0][:, others]).mean()


def test_channel_constant_over_a_window_is_exact(oracle):
    rng = np.random.default_rng(2)
    K = _rows(rng, 1, 16, 1, 64)
    K[0, :, 0, 3] = np.float16(-2.75)
    pc = oracle.PerChannelKCache(1, 1, 1)
    pc.append(K, _rows(rng, 1, 16, 1, 64), np.full((1, 16), 4, np.uint8))
    state, kc, khat, chan = pc.key_state()
    assert np.all(khat[0, :, 0, 3] == np.float32(-2.75))
    assert chan[(0, 0, 4, 0)][3, 0] == 0 and chan[(0, 0, 4, 0)][3, 1] == np.float16(-2.75).view(np.uint16)
