"""Pins for the oracle's fp16 conversions, quantizer and slot assignment (CPU only)."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quant_rows.txt")
U = 2.0 ** -24


# ---------------------------------------------------------------- fp16 <-> fp32

def test_half_to_float_all_patterns(oracle):
    h = np.arange(65536, dtype=np.uint16)
    got = oracle.half_to_float(h)
    want = h.view(np.float16).astype(np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_float_to_half_round_trip_all_patterns(oracle):
    h = np.arange(65536, dtype=np.uint16)
    f = h.view(np.float16).astype(np.float32)
    ok = ~np.isnan(f)
    assert np.array_equal(oracle.float_to_half(f)[ok], h[ok])


def test_float_to_half_ties_and_random_against_numpy(oracle):
    rng = np.random.default_rng(1)
    h = np.arange(0, 0x7BFF, dtype=np.uint16)          # finite positives below the maximum
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)           # exact halfway points (fit fp32)
    for vals in (mid, np.nextafter(mid, np.float32(np.inf)), np.nextafter(mid, np.float32(-np.inf)),
                 -mid):
        assert np.array_equal(oracle.float_to_half(vals), vals.astype(np.float16).view(np.uint16))
    r = (rng.standard_normal(200000) * np.exp(rng.uniform(-20, 12, 200000))).astype(np.float32)
    assert np.array_equal(oracle.float_to_half(r), r.astype(np.float16).view(np.uint16))
    edge = np.array([65504.0, 65519.99, 65520.0, 1e6, np.inf, -np.inf, 2.0 ** -25,
                     np.nextafter(np.float32(2.0 ** -25), np.float32(1)), 0.0, -0.0], np.float32)
    assert np.array_equal(oracle.float_to_half(edge), edge.astype(np.float16).view(np.uint16))


# ---------------------------------------------------------------- golden rows

def _parse_value(tok):
    if tok.endswith("u"):
        return float(tok[:-1]) * U
    return float(tok)


def _parse_codes(text):
    out = bytearray()
    for part in text.split():
        if "*" in part:
            hx, n = part.split("*")
            out += bytes.fromhex(hx) * int(n)
        else:
            out += bytes.fromhex(part)
    return np.frombuffer(bytes(out), dtype=np.uint8)


def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, bits, vals, mode, s_hex, z_hex, codes = [p.strip() for p in line.split("|")]
            v = [_parse_value(t) for t in vals.split()]
            if mode == "cycle":
                x = [v[i % len(v)] for i in range(64)]
            else:
                pad = _parse_value(mode.split(":")[1])
                x = v + [pad] * (64 - len(v))
            x16 = np.array(x, dtype=np.float64).astype(np.float16)
            assert np.array_equal(x16.astype(np.float64), np.array(x)), name  # fixture is exact fp16
            rows.append((name, int(bits), x16, int(s_hex, 16), int(z_hex, 16), _parse_codes(codes)))
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: r[0])
def test_quantize_row_golden(oracle, row):
    name, bits, x16, s_bits, z_bits, codes = row
    got_codes, meta = oracle.quantize_row(x16, bits)
    assert codes.size == 64 * bits // 8
    assert meta[0] == s_bits, "%s scale %04x" % (name, meta[0])
    assert meta[1] == z_bits, "%s zero-point %04x" % (name, meta[1])
    assert np.array_equal(got_codes, codes), name


def test_grid_rows_dequantize_exactly(oracle):
    """Rows that already lie on a power-of-two grid come back unchanged (xhat == x)."""
    for name, bits, x16, *_ in _golden_rows():
        if name.startswith("grid") or name in ("const4", "zeros8"):
            codes, meta = oracle.quantize_row(x16, bits)
            xhat = oracle.dequantize_row(codes, meta, 64, bits)
            assert np.array_equal(xhat, x16.astype(np.float32)), name


# ---------------------------------------------------------------- invariants

def _random_rows(rng, n, outliers=True):
    x = rng.standard_normal((n, 64)).astype(np.float32)
    if outliers:
        x[:, rng.choice(64, 4, replace=False)] *= 8
    return x.astype(np.float16)


def _unpack(codes, bits):
    """Independent unpacking: little-endian bit stream, element i = bits [i*b, i*b+b)."""
    bitstream = np.unpackbits(codes, bitorder="little")
    w = (1 << np.arange(bits)).astype(np.int64)
    return bitstream.reshape(-1, bits).astype(np.int64) @ w


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_quantizer_invariants(oracle, bits):
    rng = np.random.default_rng(bits)
    levels = (1 << bits) - 1
    for x16 in _random_rows(rng, 300):
        x = x16.astype(np.float64)
        codes, meta = oracle.quantize_row(x16, bits)
        c = _unpack(codes, bits)
        assert c.min() >= 0 and c.max() <= levels
        s = float(np.array(meta[0], np.uint16).view(np.float16))
        zp = float(np.array(meta[1], np.uint16).view(np.float16))
        # zero-point is the row minimum, an input value; scale is the fp16 rounding of range/levels
        assert zp == x.min()
        s_exact = (x.max() - x.min()) / levels
        assert s == float(np.float16(np.float32(s_exact)))
        # the minimum gets code 0 and the maximum the top code (normal scales)
        assert c[np.argmin(x)] == 0 and c[np.argmax(x)] == levels
        # dequantization error <= scale/2, up to fp32 rounding of the steps
        xhat = oracle.dequantize_row(codes, meta, 64, bits).astype(np.float64)
        slack = s * levels * 2.0 ** -11 + 1e-6       # scale rounding drifts across the range
        assert np.all(np.abs(xhat - x) <= s / 2 + slack)
        # and xhat is what the definition says, evaluated in wide precision
        assert np.allclose(xhat, c * s + zp, rtol=1e-6, atol=1e-7)
        # codes are the nearest grid index for the stored scale (away from ties)
        pos = (x - zp) / s
        frac = np.abs(pos - np.floor(pos) - 0.5)
        clear = frac > 1e-4
        assert np.array_equal(c[clear], np.clip(np.rint(pos[clear]), 0, levels).astype(np.int64))


def test_fp16_rows_round_trip_exactly(oracle):
    rng = np.random.default_rng(7)
    for x16 in _random_rows(rng, 50):
        codes, meta = oracle.quantize_row(x16, 16)
        assert codes.tobytes() == x16.astype("<f2").tobytes()
        assert meta[0] == 0 and meta[1] == 0
        xhat = oracle.dequantize_row(codes, meta, 64, 16)
        assert np.array_equal(xhat, x16.astype(np.float32))
    # every finite pattern survives
    allh = np.arange(65536, dtype=np.uint16)
    allh = allh[np.isfinite(allh.view(np.float16))]
    for chunk in allh[: (allh.size // 64) * 64].reshape(-1, 64)[::16]:
        codes, meta = oracle.quantize_row(chunk, 16)
        assert np.array_equal(codes.view("<u2"), chunk)


def test_append_matches_row_calls_and_shares_bits_between_k_and_v(oracle):
    """Eq. 24: the token's bit-width is applied to its key row and to its value row alike."""
    rng = np.random.default_rng(3)
    B, n, H = 2, 37, 3
    K = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    bits = rng.choice(np.array([2, 4, 8, 16], np.uint8), size=(B, n))
    kc, km, vc, vm = oracle.append(K, V, bits)
    for b in range(B):
        for t in range(0, n, 5):
            for h in range(H):
                for rows, codes, meta in ((K, kc, km), (V, vc, vm)):
                    c1, m1 = oracle.quantize_row(rows[b, t, h], int(bits[b, t]))
                    nb = 64 * int(bits[b, t]) // 8
                    assert np.array_equal(codes[b, t, h, :nb], c1)
                    assert not codes[b, t, h, nb:].any()
                    assert np.array_equal(meta[b, t, h], m1)


# ---------------------------------------------------------------- slots

def test_slot_assignment_is_a_bijection_per_pool(oracle):
    rng = np.random.default_rng(5)
    bits = rng.choice(np.array([2, 4, 8, 16], np.uint8), size=1000, p=[.4, .35, .2, .05])
    ps1, counts1 = oracle.assign_slots(bits[:600])
    ps2, counts = oracle.assign_slots(bits[600:], counts1)       # counts carry across calls
    ps = np.concatenate([ps1, ps2])
    pool, slot = ps >> 30, ps & 0x3FFFFFFF
    cls = np.array([{2: 0, 4: 1, 8: 2, 16: 3}[int(b)] for b in bits])
    assert np.array_equal(pool, cls)                            # class map {2,4,8,16} <-> {0..3}
    assert counts.sum() == 1000
    for p in range(4):
        s = slot[pool == p]
        assert np.array_equal(s, np.arange(s.size))             # dense, increasing with position
        assert counts[p] == s.size
    with pytest.raises(ValueError):
        oracle.assign_slots(np.array([2, 3], np.uint8))


def test_grouped_scales_reduce_to_the_row_quantizer_and_tighten_the_error(oracle):
    """Two scale groups per row: each 32-channel group is quantized exactly as a 32-element row would be (codes
    back to back, one {scale, zero-point} pair per group); with one group the cache equals the plain one and its
    attention equals the C routine's; the per-element error bound s/2 now holds per group, and the mean error does
    not grow."""
    rng = np.random.default_rng(44)
    B, Hq, H, n = 2, 4, 2, 40
    K = (rng.standard_normal((B, n, H, 64)) * 2).astype(np.float16)
    K[..., 5] *= np.float16(8.0)                                   # an outlier channel in the first group only
    V = rng.standard_normal((B, n, H, 64)).astype(np.float16)
    bits = np.array([2, 4, 8, 16], np.uint8)[rng.choice(4, size=(B, n))]
    Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
    plain = oracle.OracleCache(B, Hq, H)
    plain.append(K, V, bits)
    g1 = oracle.GroupedOracleCache(B, Hq, H, groups=1)
    g1.append(K, V, bits)
    assert np.array_equal(g1.kc, plain.kc) and np.array_equal(g1.km, plain.km) and np.array_equal(g1.vc, plain.vc)
    a, b_ = g1.decode_attn(Q).view(np.float16).astype(np.float64), plain.decode_attn(Q).view(np.float16).astype(np.float64)
    assert np.max(np.abs(a - b_)) <= 1e-3                          # same numbers up to the last fp16 rounding
    g2 = oracle.GroupedOracleCache(B, Hq, H, groups=2)
    g2.append(K, V, bits)
    assert np.array_equal(g2.pool_slot, plain.pool_slot)
    for b in range(B):
        for t in range(n):
            bt = int(bits[b, t])
            for h in range(H):
                for g in range(2):
                    codes, meta = oracle.quantize_row(K[b, t, h, 32 * g:32 * g + 32], bt)
                    gb = 32 * bt // 8
                    assert np.array_equal(g2.kc[b, t, h, g * gb:(g + 1) * gb], codes)
                    if bt < 16:
                        assert np.array_equal(g2.km[b, t, h, 2 * g:2 * g + 2], meta)
                        sf = float(oracle.half_to_float(meta[:1])[0])
                        err = np.abs(g2.khat[b, t, h, 32 * g:32 * g + 32].astype(np.float64) -
                                     K[b, t, h, 32 * g:32 * g + 32].astype(np.float64))
                        assert np.all(err <= 0.5 * sf * (1 + 2 ** -9) + 1e-6)
    q = bits < 16
    e1 = np.abs(g1.khat.astype(np.float64) - K.astype(np.float64))[q].mean()
    e2 = np.abs(g2.khat.astype(np.float64) - K.astype(np.float64))[q].mean()
    assert e2 < e1                                                 # the outlier no longer stretches the second group's grid
