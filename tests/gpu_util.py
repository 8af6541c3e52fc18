"""Helpers for the GPU parity tests: drive the C ABI through the binding with torch tensors for
device memory, and compare the store and the attention output with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2604_04722_b200 import binding as kq

DEV = "cuda:0"
# attention tolerance: |gpu - oracle| <= ATOL + RTOL * |oracle|, fp16 output, fp32 accumulation
ATOL, RTOL = 2e-3, 1e-2


def dev(a: np.ndarray) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).to(DEV)
    if a.dtype == np.uint32:
        return torch.from_numpy(a.view(np.int32)).to(DEV)
    return torch.from_numpy(a).to(DEV)


class GpuCache:
    """A kvq handle plus the shapes needed to size export buffers."""

    def __init__(self, layers, batch, q_heads, kv_heads, max_ctx, head_dim=64, scale_groups=1, arena_bytes=0,
                 k_per_channel=False):
        self.L, self.B, self.Hq, self.Hkv, self.max_ctx = layers, batch, q_heads, kv_heads, max_ctx
        self.G = scale_groups
        if k_per_channel:
            self.ctx = kq.kvq_create_perchannel(layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes)
        elif scale_groups == 1 and arena_bytes == 0:
            self.ctx = kq.kvq_create(layers, q_heads, kv_heads, head_dim, max_ctx, batch)
        else:
            self.ctx = kq.kvq_create_grouped(layers, q_heads, kv_heads, head_dim, max_ctx, batch, arena_bytes,
                                             scale_groups)

    def close(self):
        if self.ctx:
            kq.kvq_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def set_controller(self, cw):
        kq.kvq_set_controller(self.ctx, cw.hidden, *cw.as_tuple())

    def select_bits(self, feats: np.ndarray, want_logits=True):
        f = dev(feats.reshape(-1, 4).astype(np.float32))
        n = f.shape[0]
        bits = torch.zeros(n, dtype=torch.uint8, device=DEV)
        logits = torch.zeros((n, 4), dtype=torch.float32, device=DEV) if want_logits else None
        kq.kvq_select_bits(self.ctx, f, n, bits, logits)
        torch.cuda.synchronize()
        return bits.cpu().numpy().reshape(feats.shape[:-1]), (logits.cpu().numpy() if want_logits else None)

    def append(self, layer, K: np.ndarray, V: np.ndarray, bits: np.ndarray):
        Kd, Vd, bd = dev(K.view(np.uint16)), dev(V.view(np.uint16)), dev(bits.astype(np.uint8))
        kq.kvq_append(self.ctx, layer, Kd, Vd, bd, K.shape[1])
        torch.cuda.synchronize()

    def append_fused(self, layer, K, V, feats):
        Kd, Vd, fd = dev(K.view(np.uint16)), dev(V.view(np.uint16)), dev(feats.astype(np.float32))
        out = torch.zeros(feats.shape[:2], dtype=torch.uint8, device=DEV)
        kq.kvq_append_fused(self.ctx, layer, Kd, Vd, fd, K.shape[1], out)
        torch.cuda.synchronize()
        return out.cpu().numpy()

    def decode(self, layer, Q: np.ndarray) -> np.ndarray:
        Qd = dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        kq.kvq_decode_attn(self.ctx, layer, Qd, O)
        torch.cuda.synchronize()
        return O.cpu().numpy().view(np.uint16)

    def export(self, layer, pos0, n):
        B, H = self.B, self.Hkv
        bits = torch.zeros((B, n), dtype=torch.uint8, device=DEV)
        ps = torch.zeros((B, n), dtype=torch.int32, device=DEV)
        kc = torch.zeros((B, n, H, 128), dtype=torch.uint8, device=DEV)
        vc = torch.zeros_like(kc)
        km = torch.zeros((B, n, H, 2 * self.G), dtype=torch.int16, device=DEV)
        vm = torch.zeros_like(km)
        kq.kvq_export_range(self.ctx, layer, pos0, n, bits, ps, kc, vc, km, vm)
        torch.cuda.synchronize()
        return (bits.cpu().numpy(), ps.cpu().numpy().view(np.uint32), kc.cpu().numpy(), vc.cpu().numpy(),
                km.cpu().numpy().view(np.uint16), vm.cpu().numpy().view(np.uint16))


NEAR_TIE_GAP = 1e-5        # decisions whose two largest logits are closer than this are listed, not asserted
NEAR_TIE_REPORTS = []      # (what, n_decisions, [(index, logits, gap, got_bits, want_bits), ...]); printed in the summary


def compare_decisions(got_bits, want_bits, want_logits, gap, what):
    """Controller decisions against the oracle's (Eq. 22-23).  Decisions whose top-two oracle logits lie
    within NEAR_TIE_GAP of each other are LISTED (index, the four logits, gap, both answers) and kept out of
    the assertion; every other decision must agree exactly.  Returns the list."""
    got, want = np.asarray(got_bits).ravel(), np.asarray(want_bits).ravel()
    gap = np.asarray(gap).ravel()
    logits = np.asarray(want_logits).reshape(-1, 4)
    near = gap < NEAR_TIE_GAP
    rows = [(int(i), [float(x) for x in logits[i]], float(gap[i]), int(got[i]), int(want[i])) for i in np.flatnonzero(near)]
    NEAR_TIE_REPORTS.append((what, int(got.size), rows))
    bad = np.flatnonzero((got != want) & ~near)
    assert bad.size == 0, "%s: %d decisions differ outside near ties, first at %d (got %d want %d, gap %.3e)" % (
        what, bad.size, bad[0], got[bad[0]], want[bad[0]], gap[bad[0]])
    return rows


def near_tie_summary_lines(max_rows=8):
    out = []
    for what, n, rows in NEAR_TIE_REPORTS:
        out.append("%s: %d decisions, %d near ties (top-two logit gap < %g)%s" % (
            what, n, len(rows), NEAR_TIE_GAP, "" if not rows else ", %d of them decided differently" % sum(r[3] != r[4] for r in rows)))
        for i, lg, g, got, want in rows[:max_rows]:
            out.append("    token %d  logits [%s]  gap %.3e  gpu %d  oracle %d" % (i, ", ".join("%.7g" % x for x in lg), g, got, want))
        if len(rows) > max_rows:
            out.append("    ... %d more" % (len(rows) - max_rows))
    return out


def assert_store_equals_oracle(gpu: GpuCache, layer: int, ocache, pos0=0, n=None):
    """Bit-exact: bit-widths, (pool, slot), packed codes, scale / zero-point."""
    n = len(ocache) - pos0 if n is None else n
    bits, ps, kc, vc, km, vm = gpu.export(layer, pos0, n)
    sl = slice(pos0, pos0 + n)
    assert np.array_equal(bits, ocache.bits[:, sl]), "bit-widths differ"
    assert np.array_equal(ps, ocache.pool_slot[:, sl]), "(pool, slot) differ"
    assert np.array_equal(km, ocache.km[:, sl]), "K scale/zero-point differ"
    assert np.array_equal(vm, ocache.vm[:, sl]), "V scale/zero-point differ"
    assert np.array_equal(kc, ocache.kc[:, sl]), "K codes differ"
    assert np.array_equal(vc, ocache.vc[:, sl]), "V codes differ"


def assert_attention_close(got_u16: np.ndarray, want_u16: np.ndarray, what=""):
    got = got_u16.view(np.float16).astype(np.float64)
    want = want_u16.view(np.float16).astype(np.float64)
    err = np.abs(got - want)
    bound = ATOL + RTOL * np.abs(want)
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert np.all(err <= bound), "%s attention mismatch: max err %.3e at %s (got %.5f want %.5f)" % (
        what, err.max(), worst, got[worst], want[worst])
    return float(err.max())
