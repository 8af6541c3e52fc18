"""ctypes front end of the plain CPU oracle (``kvq_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  Nothing in the CUDA package imports it, and it
imports nothing from the CUDA package.

All arithmetic lives in the C file; this module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvq_oracle.c")
_LIB = os.path.join(_HERE, "libkvq_oracle.so")

CFLAGS = ["-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_half_to_float.restype = C.c_float
        _lib.oracle_half_to_float.argtypes = [C.c_uint16]
        _lib.oracle_float_to_half.restype = C.c_uint16
        _lib.oracle_float_to_half.argtypes = [C.c_float]
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def _u16(a) -> np.ndarray:
    """fp16 arrays are passed as their bit patterns."""
    a = np.asarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    return np.ascontiguousarray(a, dtype=np.uint16)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def half_to_float(h: np.ndarray) -> np.ndarray:
    h = _u16(h)
    out = np.empty(h.shape, dtype=np.float32)
    lib().oracle_half_to_float_array(_p(h), C.c_int(h.size), _p(out))
    return out


def float_to_half(f: np.ndarray) -> np.ndarray:
    f = _c(f, np.float32)
    out = np.empty(f.shape, dtype=np.uint16)
    lib().oracle_float_to_half_array(_p(f), C.c_int(f.size), _p(out))
    return out


def select_bits(feats, hidden, W1, b1, W2, b2, W3, b3
                ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Controller decision for feats [..., 4] -> (bits u8 [...], logits [...,4], gap [...])."""
    feats = _c(feats, np.float32)
    shape = feats.shape[:-1]
    n = int(np.prod(shape)) if shape else 1
    W1, b1, W2, b2, W3, b3 = (_c(x, np.float32) for x in (W1, b1, W2, b2, W3, b3))
    assert W1.shape == (hidden, 4) and W2.shape == (hidden, hidden) and W3.shape == (4, hidden)
    bits = np.empty(n, dtype=np.uint8)
    logits = np.empty((n, 4), dtype=np.float32)
    gap = np.empty(n, dtype=np.float32)
    rc = lib().oracle_select_bits(_p(feats), C.c_int(n), C.c_int(hidden),
                                  _p(W1), _p(b1), _p(W2), _p(b2), _p(W3), _p(b3),
                                  _p(bits), _p(logits), _p(gap))
    if rc != 0:
        raise ValueError("oracle_select_bits failed: %d" % rc)
    return bits.reshape(shape), logits.reshape(shape + (4,)), gap.reshape(shape)


def assign_slots(bits, counts: Optional[np.ndarray] = None
                 ) -> Tuple[np.ndarray, np.ndarray]:
    """(pool<<30 | slot) for one sequence's tokens in position order; returns (pool_slot, counts)."""
    bits = _c(bits, np.uint8)
    counts = np.zeros(4, dtype=np.uint32) if counts is None else _c(counts, np.uint32).copy()
    ps = np.empty(bits.shape[0], dtype=np.uint32)
    rc = lib().oracle_assign_slots(_p(bits), C.c_int(bits.shape[0]), _p(counts), _p(ps))
    if rc != 0:
        raise ValueError("oracle_assign_slots failed: %d" % rc)
    return ps, counts


def quantize_row(x, bits: int) -> Tuple[np.ndarray, np.ndarray]:
    """One fp16 row -> (codes u8 [D*bits/8], meta u16 [2] = {scale, zero-point} bit patterns)."""
    x = _u16(x)
    D = x.shape[0]
    codes = np.zeros(D * bits // 8, dtype=np.uint8)
    meta = np.zeros(2, dtype=np.uint16)
    rc = lib().oracle_quantize_row(_p(x), C.c_int(D), C.c_int(bits), _p(codes), _p(meta))
    if rc != 0:
        raise ValueError("oracle_quantize_row failed: %d" % rc)
    return codes, meta


def dequantize_row(codes, meta, D: int, bits: int) -> np.ndarray:
    codes = _c(codes, np.uint8)
    meta = _c(meta, np.uint16)
    out = np.empty(D, dtype=np.float32)
    rc = lib().oracle_dequantize_row(_p(codes), _p(meta), C.c_int(D), C.c_int(bits), _p(out))
    if rc != 0:
        raise ValueError("oracle_dequantize_row failed: %d" % rc)
    return out


def append(K, V, bits):
    """K, V fp16 [B][n][Hkv][D], bits u8 [B][n] -> (kcodes, kmeta, vcodes, vmeta).

    codes u8 [B][n][Hkv][2*D] (row stride 2*D, tail zero), meta u16 [B][n][Hkv][2].
    """
    K, V = _u16(K), _u16(V)
    bits = _c(bits, np.uint8)
    B, n, H, D = K.shape
    assert V.shape == K.shape and bits.shape == (B, n)
    kc = np.empty((B, n, H, 2 * D), dtype=np.uint8)
    vc = np.empty((B, n, H, 2 * D), dtype=np.uint8)
    km = np.empty((B, n, H, 2), dtype=np.uint16)
    vm = np.empty((B, n, H, 2), dtype=np.uint16)
    rc = lib().oracle_append(_p(K), _p(V), _p(bits), C.c_int(B), C.c_int(n), C.c_int(H),
                             C.c_int(D), _p(kc), _p(km), _p(vc), _p(vm))
    if rc != 0:
        raise ValueError("oracle_append failed: %d" % rc)
    return kc, km, vc, vm


def decode_attn(Q, q_heads: int, kv_heads: int, bits, kc, km, vc, vm,
                want64: bool = False):
    """Q fp16 [B][Hq][D] over the cache written by ``append`` -> O fp16 bit patterns [B][Hq][D]."""
    Q = _u16(Q)
    B, Hq, D = Q.shape
    bits = _c(bits, np.uint8)
    n = bits.shape[1]
    kc, vc = _c(kc, np.uint8), _c(vc, np.uint8)
    km, vm = _c(km, np.uint16), _c(vm, np.uint16)
    assert Hq == q_heads and kc.shape == (B, n, kv_heads, 2 * D)
    out = np.empty((B, Hq, D), dtype=np.uint16)
    out64 = np.empty((B, Hq, D), dtype=np.float64) if want64 else None
    rc = lib().oracle_decode_attn(_p(Q), C.c_int(B), C.c_int(q_heads), C.c_int(kv_heads),
                                  C.c_int(D), C.c_int(n), _p(bits), _p(kc), _p(km),
                                  _p(vc), _p(vm), _p(out), _p(out64))
    if rc != 0:
        raise ValueError("oracle_decode_attn failed: %d" % rc)
    return (out, out64) if want64 else out


def decode_probs(Q, q_heads: int, kv_heads: int, bits, kc, km, vc, vm) -> np.ndarray:
    """The attention weights of ``decode_attn``: fp64 [B][Hq][n]."""
    Q = _u16(Q)
    B, Hq, D = Q.shape
    bits = _c(bits, np.uint8)
    n = bits.shape[1]
    kc, vc = _c(kc, np.uint8), _c(vc, np.uint8)
    km, vm = _c(km, np.uint16), _c(vm, np.uint16)
    probs = np.empty((B, Hq, n), dtype=np.float64)
    rc = lib().oracle_decode_probs(_p(Q), C.c_int(B), C.c_int(q_heads), C.c_int(kv_heads), C.c_int(D), C.c_int(n),
                                   _p(bits), _p(kc), _p(km), _p(vc), _p(vm), _p(probs))
    if rc != 0:
        raise ValueError("oracle_decode_probs failed: %d" % rc)
    return probs


# ---- token-level saliency features (Section 3.2), plain fp64 numpy from the definitions

def token_entropy(logits) -> np.ndarray:
    """Eq. 14: H_t = -sum_v p_t(v) log p_t(v), p_t = Softmax(z_t); logits [n][V] -> [n] (natural log)."""
    z = np.asarray(logits, dtype=np.float64)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(p > 0, p * np.log(p), 0.0)
    return -t.sum(axis=1)


def token_confidence(logits) -> np.ndarray:
    """The confidence term C_t of Eq. 17, which the paper names without defining: taken as the largest
    next-token probability, max_v Softmax(z_t)_v."""
    z = np.asarray(logits, dtype=np.float64)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    return (p / p.sum(axis=1, keepdims=True)).max(axis=1)


def token_rarity(token_ids, counts, total: int, observed: int) -> np.ndarray:
    """Eq. 15: R_t = -log((c(x_t) + 1) / (N + |V_obs| + 1)); counts [V] running counts, total = N."""
    c = np.asarray(counts, dtype=np.float64)[np.asarray(token_ids, dtype=np.int64)]
    return -np.log((c + 1.0) / (float(total) + float(observed) + 1.0))


def attention_variance(probs) -> np.ndarray:
    """Eq. 16: V_t = (1/h) sum_i Var(A_i), with Var taken over the cached positions the query row of head i
    attends to (population variance); probs [B][h][n] -> [B]."""
    return np.var(np.asarray(probs, dtype=np.float64), axis=2).mean(axis=1)


class OracleCache:
    """Position-ordered mixed-precision cache of one layer: append rows, then attend."""

    def __init__(self, batch: int, q_heads: int, kv_heads: int, head_dim: int = 64):
        self.B, self.Hq, self.Hkv, self.D = batch, q_heads, kv_heads, head_dim
        self.bits = np.zeros((batch, 0), dtype=np.uint8)
        self.kc = np.zeros((batch, 0, kv_heads, 2 * head_dim), dtype=np.uint8)
        self.vc = np.zeros_like(self.kc)
        self.km = np.zeros((batch, 0, kv_heads, 2), dtype=np.uint16)
        self.vm = np.zeros_like(self.km)
        self.counts = np.zeros((batch, 4), dtype=np.uint32)
        self.pool_slot = np.zeros((batch, 0), dtype=np.uint32)

    def __len__(self) -> int:
        return self.bits.shape[1]

    def append(self, K, V, bits) -> None:
        bits = _c(bits, np.uint8)
        kc, km, vc, vm = append(K, V, bits)
        ps = np.empty(bits.shape, dtype=np.uint32)
        for b in range(self.B):
            ps[b], self.counts[b] = assign_slots(bits[b], self.counts[b])
        self.bits = np.concatenate([self.bits, bits], axis=1)
        self.kc = np.concatenate([self.kc, kc], axis=1)
        self.vc = np.concatenate([self.vc, vc], axis=1)
        self.km = np.concatenate([self.km, km], axis=1)
        self.vm = np.concatenate([self.vm, vm], axis=1)
        self.pool_slot = np.concatenate([self.pool_slot, ps], axis=1)

    def decode_attn(self, Q, want64: bool = False):
        return decode_attn(Q, self.Hq, self.Hkv, self.bits, self.kc, self.km,
                           self.vc, self.vm, want64=want64)

    def decode_probs(self, Q) -> np.ndarray:
        return decode_probs(Q, self.Hq, self.Hkv, self.bits, self.kc, self.km, self.vc, self.vm)

    def attend_last(self, Q):
        """Causal attention of the last T cached positions (Eq. 5 at each of them): Q fp16 [B][T][Hq][D];
        row i sees the first len - T + i + 1 tokens.  Written as T plain calls on truncated caches."""
        Q = _u16(Q)
        B, T, Hq, D = Q.shape
        n = len(self)
        assert 1 <= T <= n
        out = np.empty((B, T, Hq, D), dtype=np.uint16)
        for i in range(T):
            m = n - T + i + 1
            out[:, i] = decode_attn(np.ascontiguousarray(Q[:, i]), self.Hq, self.Hkv, self.bits[:, :m],
                                    self.kc[:, :m], self.km[:, :m], self.vc[:, :m], self.vm[:, :m])
        return out


class GroupedOracleCache:
    """The same cache with finer scale granularity: every row is cut into ``groups`` groups of
    head_dim / groups consecutive channels and the row quantizer (the reading of Q_b in Eq. 24) is applied to
    each group on its own, so a row carries ``groups`` {scale, zero-point} pairs.  Canonical form: the codes of
    the groups back to back (element order unchanged), meta u16 [..][2 * groups].  Attention is Eq. 5 by its
    definition (fp64) over the dequantized rows."""

    def __init__(self, batch: int, q_heads: int, kv_heads: int, groups: int = 2, head_dim: int = 64):
        assert head_dim % groups == 0
        self.B, self.Hq, self.Hkv, self.D, self.G = batch, q_heads, kv_heads, head_dim, groups
        self.bits = np.zeros((batch, 0), dtype=np.uint8)
        self.kc = np.zeros((batch, 0, kv_heads, 2 * head_dim), dtype=np.uint8)
        self.vc = np.zeros_like(self.kc)
        self.km = np.zeros((batch, 0, kv_heads, 2 * groups), dtype=np.uint16)
        self.vm = np.zeros_like(self.km)
        self.khat = np.zeros((batch, 0, kv_heads, head_dim), dtype=np.float32)
        self.vhat = np.zeros_like(self.khat)
        self.counts = np.zeros((batch, 4), dtype=np.uint32)
        self.pool_slot = np.zeros((batch, 0), dtype=np.uint32)

    def __len__(self) -> int:
        return self.bits.shape[1]

    def _one(self, X, bits):
        B, n, H, D = X.shape
        G, Dg = self.G, D // self.G
        Xg = np.ascontiguousarray(_u16(X).reshape(B, n, H * G, Dg))
        cg, mg, _, _ = append(Xg, Xg, bits)                       # group rows: codes [B][n][H*G][2*Dg], meta [..][2]
        codes = np.zeros((B, n, H, 2 * D), dtype=np.uint8)
        hat = np.zeros((B, n, H, D), dtype=np.float32)
        for b in range(B):
            for t in range(n):
                bt = int(bits[b, t])
                gb = Dg * bt // 8
                for h in range(H):
                    for g in range(G):
                        codes[b, t, h, g * gb:(g + 1) * gb] = cg[b, t, h * G + g, :gb]
                        hat[b, t, h, g * Dg:(g + 1) * Dg] = dequantize_row(cg[b, t, h * G + g, :gb], mg[b, t, h * G + g], Dg, bt)
        return codes, mg.reshape(B, n, H, 2 * G), hat

    def append(self, K, V, bits) -> None:
        bits = _c(bits, np.uint8)
        kc, km, kh = self._one(K, bits)
        vc, vm, vh = self._one(V, bits)
        ps = np.empty(bits.shape, dtype=np.uint32)
        for b in range(self.B):
            ps[b], self.counts[b] = assign_slots(bits[b], self.counts[b])
        self.bits = np.concatenate([self.bits, bits], axis=1)
        self.kc = np.concatenate([self.kc, kc], axis=1)
        self.vc = np.concatenate([self.vc, vc], axis=1)
        self.km = np.concatenate([self.km, km], axis=1)
        self.vm = np.concatenate([self.vm, vm], axis=1)
        self.khat = np.concatenate([self.khat, kh], axis=1)
        self.vhat = np.concatenate([self.vhat, vh], axis=1)
        self.pool_slot = np.concatenate([self.pool_slot, ps], axis=1)

    def decode_attn(self, Q) -> np.ndarray:
        """fp16 bit patterns [B][Hq][D]: Softmax(q K^T / sqrt(D)) V over the dequantized rows, in fp64."""
        q = half_to_float(_u16(Q)).astype(np.float64)
        g = self.Hq // self.Hkv
        out = np.empty((self.B, self.Hq, self.D), dtype=np.float64)
        for b in range(self.B):
            for h in range(self.Hq):
                k = self.khat[b, :, h // g].astype(np.float64)
                v = self.vhat[b, :, h // g].astype(np.float64)
                z = k @ q[b, h] / np.sqrt(float(self.D))
                p = np.exp(z - z.max())
                p /= p.sum()
                out[b, h] = p @ v
        return np.asarray(out, dtype=np.float16).view(np.uint16)          # fp64 -> fp16, round to nearest even


def _unpack_codes(codes: np.ndarray, n: int, bits: int) -> np.ndarray:
    """The first n codes of little-endian linear packed rows: codes u8 [..., bytes] -> u8 [..., n]."""
    idx = np.arange(n) * bits
    return (codes[..., idx // 8] >> (idx % 8).astype(np.uint8)) & np.uint8((1 << bits) - 1)


def _pack_codes(c: np.ndarray, bits: int, row_bytes: int) -> np.ndarray:
    """Codes u8 [..., n] -> little-endian linear packed rows u8 [..., row_bytes] (tail zero)."""
    n = c.shape[-1]
    out = np.zeros(c.shape[:-1] + (row_bytes,), dtype=np.uint8)
    for i in range(n):
        bp = i * bits
        out[..., bp // 8] |= (c[..., i].astype(np.uint8) << np.uint8(bp % 8))
    return out


class PerChannelKCache:
    """A cache whose KEYS are quantized per channel instead of per token (the granularity of the key quantizers in
    the related work the paper cites in Section 2), values per token as in ``OracleCache``.

    Reading.  Tokens go to the pool of their bit-width and take slots in position order as before.  The slots of a
    (sequence, KV head, precision) stream are cut into WINDOWS of ``window`` = 16 consecutive slots.  In a complete
    window every channel is a row for the row quantizer (the reading of Q_b in Eq. 24): its ``window`` key values,
    one per token, get one {scale, zero-point} pair and codes by the same arithmetic.  The stream's last, still
    incomplete window keeps its key rows in fp16 (they are quantized when the window fills); 16-bit tokens keep
    fp16 rows as always.  Attention is Eq. 5 by its definition (fp64) over the dequantized rows.

    Kept per token and KV head, for comparison with other implementations: ``k_state`` 0 = fp16 row (16-bit class or
    open window), 1 = packed; ``kc`` the canonical row (packed codes in element order, or the fp16 row); per
    (stream, window, channel) ``chan_meta`` {scale, zero-point} bit patterns."""

    def __init__(self, batch: int, q_heads: int, kv_heads: int, head_dim: int = 64, window: int = 16):
        self.B, self.Hq, self.Hkv, self.D, self.W = batch, q_heads, kv_heads, head_dim, window
        self.bits = np.zeros((batch, 0), dtype=np.uint8)
        self.K = np.zeros((batch, 0, kv_heads, head_dim), dtype=np.uint16)      # fp16 bit patterns as appended
        self.vc = np.zeros((batch, 0, kv_heads, 2 * head_dim), dtype=np.uint8)
        self.vm = np.zeros((batch, 0, kv_heads, 2), dtype=np.uint16)
        self.counts = np.zeros((batch, 4), dtype=np.uint32)
        self.pool_slot = np.zeros((batch, 0), dtype=np.uint32)

    def __len__(self) -> int:
        return self.bits.shape[1]

    def append(self, K, V, bits) -> None:
        bits = _c(bits, np.uint8)
        _, _, vc, vm = append(V, V, bits)                          # values: the per-token row quantizer
        ps = np.empty(bits.shape, dtype=np.uint32)
        for b in range(self.B):
            ps[b], self.counts[b] = assign_slots(bits[b], self.counts[b])
        self.bits = np.concatenate([self.bits, bits], axis=1)
        self.K = np.concatenate([self.K, _u16(K)], axis=1)
        self.vc = np.concatenate([self.vc, vc], axis=1)
        self.vm = np.concatenate([self.vm, vm], axis=1)
        self.pool_slot = np.concatenate([self.pool_slot, ps], axis=1)

    def key_state(self):
        """(k_state u8 [B][n][Hkv], kc u8 [B][n][Hkv][2D], khat f32 [B][n][Hkv][D], chan_meta {(b, h, bits, window):
        u16 [D][2]}) of the cache as it stands."""
        B, n, H, D, W = self.B, len(self), self.Hkv, self.D, self.W
        k_state = np.zeros((B, n, H), dtype=np.uint8)
        kc = np.zeros((B, n, H, 2 * D), dtype=np.uint8)
        khat = half_to_float(self.K)
        kc[..., 0:2 * D:2] = (self.K & 0xFF).astype(np.uint8)          # fp16 rows, little-endian
        kc[..., 1:2 * D:2] = (self.K >> 8).astype(np.uint8)
        chan_meta = {}
        for b in range(B):
            for bt in (2, 4, 8):
                pos = np.flatnonzero(self.bits[b] == bt)               # position order = slot order
                for w in range(len(pos) // W):
                    p = pos[w * W:(w + 1) * W]
                    for h in range(H):
                        # every channel's W values as one row of the row quantizer: [1][1][D][W]
                        rows = np.ascontiguousarray(self.K[b, p, h, :].T)[None, None]
                        cg, mg, _, _ = append(rows, rows, np.full((1, 1), bt, np.uint8))
                        codes = _unpack_codes(cg[0, 0, :, :W * bt // 8], W, bt)       # [D][W]
                        kc[b, p, h, :] = _pack_codes(np.ascontiguousarray(codes.T), bt, 2 * D)
                        k_state[b, p, h] = 1
                        chan_meta[(b, h, bt, w)] = mg[0, 0]
                        for i in range(D):
                            khat[b, p, h, i] = dequantize_row(cg[0, 0, i, :W * bt // 8], mg[0, 0, i], W, bt)
        return k_state, kc, khat, chan_meta

    def decode_attn(self, Q) -> np.ndarray:
        """fp16 bit patterns [B][Hq][D]: Softmax(q K^T / sqrt(D)) V over the dequantized rows, in fp64."""
        _, _, khat, _ = self.key_state()
        q = half_to_float(_u16(Q)).astype(np.float64)
        g = self.Hq // self.Hkv
        out = np.empty((self.B, self.Hq, self.D), dtype=np.float64)
        n = len(self)
        for b in range(self.B):
            vhat = np.empty((n, self.Hkv, self.D), dtype=np.float64)
            for t in range(n):
                bt = int(self.bits[b, t])
                for h in range(self.Hkv):
                    vhat[t, h] = dequantize_row(self.vc[b, t, h, :self.D * bt // 8], self.vm[b, t, h], self.D, bt)
            for h in range(self.Hq):
                k = khat[b, :, h // g].astype(np.float64)
                z = k @ q[b, h] / np.sqrt(float(self.D))
                p = np.exp(z - z.max())
                p /= p.sum()
                out[b, h] = p @ vhat[:, h // g]
        return np.asarray(out, dtype=np.float16).view(np.uint16)
