"""Seeded random shapes through the whole path against the oracle: batch, head counts and grouping,
cached length (zero included), bit mix (degenerate mixes included), split count, scale granularity
and controller width are drawn per case; a prefill (bit-widths given or decided by the controller),
then decode steps through kvq_decode_step, then kvq_decode_attn and its fixed-scratch variant.
Decisions and the store are compared bit for bit, every attention output within the tolerance."""
import os

import numpy as np
import pytest

from paper_2604_04722_b200 import synth

pytestmark = pytest.mark.gpu

BITS = np.array([2, 4, 8, 16], dtype=np.uint8)
CASES = int(os.environ.get("KVQ_RANDOM_CASES", "36"))    # more seeds for a longer soak


@pytest.fixture(scope="module")
def gu():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_04722_b200 import build
    build.build()
    import gpu_util
    return gpu_util


def _draw(seed):
    rng = np.random.default_rng(1000 + seed)
    case = {
        "B": int(rng.integers(1, 5)),
        "Hkv": int(rng.choice([1, 2, 3, 5, 8, 17])),
        "group": int(rng.choice([1, 1, 2, 3, 4])),
        "n": int(rng.choice([0, 1, 15, 16, 17, 100, 255, 256, 257, 700, 1633, 2500])),
        "steps": int(rng.integers(1, 7)),
        "splits": int(rng.choice([0, 0, 0, 1, 2, 3, 5, 16, 64])),
        "layout": str(rng.choice(["row", "row", "row", "row", "two groups", "per-channel keys"])),
        "hidden": int(rng.choice([32, 32, 32, 7, 128])),
        "fused_prefill": bool(rng.integers(0, 2)),
        "kscale": float(rng.choice([0.05, 1.0, 1.0, 6.0])),
    }
    p = rng.dirichlet([0.6, 0.6, 0.6, 0.6])
    if rng.integers(0, 4) == 0:                      # a degenerate mix: one or two classes only
        p = np.zeros(4)
        for k in rng.choice(4, size=int(rng.integers(1, 3)), replace=False):
            p[k] = 1.0
        p /= p.sum()
    case["mix"] = p
    return rng, case


@pytest.mark.parametrize("seed", range(CASES))
def test_random_shape(gu, oracle, seed):
    import torch
    from paper_2604_04722_b200 import binding as kq
    rng, c = _draw(seed)
    B, H, Hq, n, steps = c["B"], c["Hkv"], c["Hkv"] * c["group"], c["n"], c["steps"]
    what = "case %d: %s" % (seed, {k: (v if k != "mix" else np.round(v, 2).tolist()) for k, v in c.items()})
    cw = synth.controller_weights(322 if c["hidden"] == 32 else 5 if c["hidden"] == 7 else 2, c["hidden"])
    if c["layout"] == "two groups":
        oc, g = oracle.GroupedOracleCache(B, Hq, H, 2), gu.GpuCache(1, B, Hq, H, n + steps, scale_groups=2)
    elif c["layout"] == "per-channel keys":
        oc, g = oracle.PerChannelKCache(B, Hq, H), gu.GpuCache(1, B, Hq, H, n + steps, k_per_channel=True)
    else:
        oc, g = oracle.OracleCache(B, Hq, H), gu.GpuCache(1, B, Hq, H, n + steps)
    with g:
        g.set_controller(cw)
        kq.kvq_set_splits(g.ctx, c["splits"])
        if n:
            K = (rng.standard_normal((B, n, H, 64)) * c["kscale"]).astype(np.float16)
            V = (rng.standard_normal((B, n, H, 64)) * c["kscale"]).astype(np.float16)
            if c["fused_prefill"]:
                feats = synth.features_batch(seed, B, 0, n)
                bits, logits, gap = oracle.select_bits(feats, cw.hidden, *cw.as_tuple())
                got = g.append_fused(0, K, V, feats)
                near = gu.compare_decisions(got, bits, logits, gap, "random shapes, prefill of case %d" % seed)
                assert all(r[3] == r[4] for r in near), what
            else:
                bits = BITS[rng.choice(4, size=(B, n), p=c["mix"])]
                g.append(0, K, V, bits)
            oc.append(K, V, bits)
        feats = synth.features_batch(seed + 500, B, n, steps)
        want_bits, want_logits, gap = oracle.select_bits(feats, cw.hidden, *cw.as_tuple())
        got_bits = np.zeros_like(want_bits)
        for s in range(steps):
            K1 = (rng.standard_normal((B, 1, H, 64)) * c["kscale"]).astype(np.float16)
            V1 = (rng.standard_normal((B, 1, H, 64)) * c["kscale"]).astype(np.float16)
            Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
            oc.append(K1, V1, want_bits[:, s:s + 1])
            Qd = gu.dev(Q.view(np.uint16))
            O = torch.zeros_like(Qd)
            bd = torch.zeros(B, dtype=torch.uint8, device=gu.DEV)
            kq.kvq_decode_step(g.ctx, 0, gu.dev(feats[:, s].astype(np.float32)), gu.dev(K1.view(np.uint16)),
                               gu.dev(V1.view(np.uint16)), Qd, O, bd)
            torch.cuda.synchronize()
            got_bits[:, s] = bd.cpu().numpy()
            gu.assert_attention_close(O.cpu().numpy().view(np.uint16), oc.decode_attn(Q), "%s, step %d" % (what, s))
        near = gu.compare_decisions(got_bits, want_bits, want_logits, gap, "random shapes, steps of case %d" % seed)
        assert all(r[3] == r[4] for r in near), what
        # attention alone over the final cache, with the handle's scratch and with the fixed array
        Q = rng.standard_normal((B, Hq, 64)).astype(np.float16)
        want = oc.decode_attn(Q)
        gu.assert_attention_close(g.decode(0, Q), want, what + ", kvq_decode_attn")
        Qd = gu.dev(Q.view(np.uint16))
        O = torch.zeros_like(Qd)
        rc = kq.lib().kvq_decode_attn_static(g.ctx, 0, Qd.data_ptr(), O.data_ptr(), None)
        assert rc in (0, kq.KVQ_ERR_TOO_LARGE), what
        if rc == 0:
            torch.cuda.synchronize()
            gu.assert_attention_close(O.cpu().numpy().view(np.uint16), want, what + ", fixed scratch")
        if c["layout"] != "per-channel keys":
            gu.assert_store_equals_oracle(g, 0, oc)
        assert kq.kvq_device_status(g.ctx) == 0, what
