#!/usr/bin/env python
"""Benchmark of the adaptive KV-cache hot path on B200.

A "step" is one pass of the whole path over one batch of synthetic input: controller decision
for the step's new tokens (Eq. 19-23), quantize-append of their K/V rows (Eq. 24, Eq. 4) and
decode attention over the whole mixed-precision cache (Eq. 5).  The workload is the stress
configuration the bandwidth target is quoted on: one SmolLM-1.7B-shaped layer, 32 query / 32 KV
heads, head_dim 64, batch 16, context 32768, bit-widths i.i.d. {2:50%, 4:30%, 8:15%, FP16:5%}.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference ...                     # the CPU oracle on a bounded sample
    python bench.py --sweep-splits                           # automatic launch plan against explicit split counts
    python bench.py --features-only                          # the on-device feature kernel alone

Timing protocol: after W warm-up steps a block of exactly K steps is timed with CUDA events between
device synchronisations (and barriers when N > 1); the block is repeated `--blocks` times (default
10) and `ms_per_step` is the median block, with the minimum and maximum beside it.

With N > 1 (launched by torchrun) every rank runs an independent replica of the workload (the
path has no exchange step); the reported value is the sum over ranks divided by the slowest
rank's device time.

Prints ONE JSON line.  `value` = algorithmic bytes of a step (packed codes + scales read by the
attention, Q/O, the new tokens' fp16 rows read and packed rows + index written, their features)
per second, inputs resident in HBM.  `e2e` = the same through kvq_decode_step_host with pinned
host buffers, copies inside the timed region.  At N = 1 the line also carries `other_workloads`:
the other four SmolLM-shaped workloads (and the uniform-precision variants of the fourth) timed
the same way with fewer steps, each with the oracle timed on a sample of it.
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
import json
import math
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_04722_b200 import synth  # noqa: E402

ROW_BYTES = {2: 40, 4: 72, 8: 136, 16: 256}          # K+V bytes per (token, KV head), scales included
METRIC = "decode_step_kv_bandwidth"
UNIT = "GB/s"
L2_BYTES = 126e6
NEAR_TIE_GAP = 1e-5
ORACLE_SAMPLE_SEQS = 2                               # whole sequences of the workload the oracle legs run

# DRAM traffic of one launch of the step kernel (ncu: dram__bytes_read.sum + dram__bytes_write.sum) is kept in a
# small text file beside the profile it comes from, together with a hash of the kernel sources it was
# captured on; when the sources have changed since, the bench prints "traffic": null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "k_decode_step_cfg5_traffic.txt")
CSRC_DIR = os.path.join(ROOT, "paper_2604_04722_b200", "csrc")


def csrc_hash() -> str:
    h = hashlib.sha256()
    for name in sorted(os.listdir(CSRC_DIR)):
        if name.endswith((".cu", ".cuh")):
            h.update(name.encode())
            with open(os.path.join(CSRC_DIR, name), "rb") as f:
                h.update(f.read())
    return h.hexdigest()


def recorded_traffic():
    """(bytes per full cfg5 launch or None, note).  The file holds `key = value` lines: csrc_sha256,
    dram_bytes_per_launch (of the captured case) and scale (rows of a full launch / rows of the captured case)."""
    try:
        kv = {}
        for line in open(TRAFFIC_FILE):
            if "=" in line and not line.lstrip().startswith("#"):
                k, v = line.split("=", 1)
                kv[k.strip()] = v.strip()
        if kv["csrc_sha256"] != csrc_hash():
            return None, "kernel sources changed since the capture in profiles/"
        return float(kv["dram_bytes_per_launch"]) * float(kv["scale"]), "ncu capture of a quarter of the sequences, x %s" % kv["scale"]
    except Exception as e:                                 # no file, or a malformed one
        return None, "no usable capture record (%s)" % type(e).__name__


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def step_bytes(wl, resident_bytes_mean, new_row_bytes_mean):
    """Algorithmic bytes of one step of one layer (per replica): (decode, append)."""
    qo = 2 * wl.batch * wl.q_heads * wl.head_dim * 2
    decode = resident_bytes_mean + qo
    append = (wl.batch * wl.kv_heads * 256            # fp16 K and V rows read
              + new_row_bytes_mean                    # packed rows written
              + wl.batch * 4                          # index words
              + wl.batch * 16)                        # features
    return decode, append


class ClockSampler:
    """nvidia-smi sampler for SM clocks and throttle reasons during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = os.path.join("/tmp", "kvq_clocks_%d_%d.csv" % (os.getpid(), gpu_index))

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, smax, power, reasons = [], [], [], set()
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1]))
                    smax.append(float(p[2]))
                    power.append(float(p[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)), samples=len(sm),
                       sm_mhz_min=float(min(sm)), power_w_max=float(max(power)) if power else None)
        out["reasons"] = sorted(reasons)
        return out


def aggregate_over_ranks(times_ms, step_bytes_this_rank, dist, device):
    """The whole job's figures from one rank's: every time becomes the slowest rank's (max), the bytes
    of a step become the sum over the ranks' replicas.  `dist` is torch.distributed or None."""
    import torch
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    nbytes = torch.tensor([float(step_bytes_this_rank)], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(nbytes, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(nbytes.item())


def oracle_sequences(wl):
    return list(range(min(ORACLE_SAMPLE_SEQS, wl.batch)))


def oracle_leg(wl, seqs, steps, warmup):
    """The CPU oracle, as it stands, on a bounded sample of the workload: `seqs` whole sequences of ONE layer.
    Each step = decision for the new tokens + quantize-append + attention over everything cached."""
    import oracle
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)
    nb = len(seqs)
    K = np.stack([synth.kv_rows(wl.seed, 0, b, 0, wl.context, wl.kv_heads)[0] for b in seqs])
    V = np.stack([synth.kv_rows(wl.seed, 0, b, 0, wl.context, wl.kv_heads)[1] for b in seqs])
    if wl.bits_mode == "controller":
        feats = np.stack([synth.features(wl.seed, b, 0, wl.context) for b in seqs])
        bits, _, _ = oracle.select_bits(feats, wl.hidden, *cw.as_tuple())
    else:
        bits = np.stack([synth.workload_bits(wl, b, 0, wl.context) for b in seqs])
    oc = oracle.OracleCache(nb, wl.q_heads, wl.kv_heads)
    t0 = time.perf_counter()
    oc.append(K, V, bits)
    prefill_s = time.perf_counter() - t0
    del K, V
    times, nbytes = [], []
    for step in range(warmup + steps):
        pos = wl.context + step
        f1 = np.stack([synth.features(wl.seed, b, pos, 1) for b in seqs])
        k1 = np.stack([synth.kv_rows(wl.seed, 0, b, pos, 1, wl.kv_heads)[0] for b in seqs])
        v1 = np.stack([synth.kv_rows(wl.seed, 0, b, pos, 1, wl.kv_heads)[1] for b in seqs])
        Q = synth.queries(wl.seed, 0, step, wl.batch, wl.q_heads)[seqs]
        t0 = time.perf_counter()
        b1, _, _ = oracle.select_bits(f1, wl.hidden, *cw.as_tuple())
        oc.append(k1, v1, b1)
        oc.decode_attn(Q)
        dt = time.perf_counter() - t0
        if step >= warmup:
            times.append(dt)
            resident = sum(ROW_BYTES[int(x)] for x in oc.bits.ravel()) * wl.kv_heads
            new_rows = sum(ROW_BYTES[int(x)] for x in b1.ravel()) * wl.kv_heads
            nbytes.append(resident + 2 * nb * wl.q_heads * 128 + nb * wl.kv_heads * 256 + new_rows + nb * 20)
    total_t = float(np.sum(times))
    return {
        "value": float(np.sum(nbytes)) / total_t / 1e9,
        "ms_per_step": 1e3 * total_t / len(times),
        "cores": oracle.num_threads(),
        "sample": "%d of %d sequences of the workload (whole sequences, every head, one of %d layers, context %d); %d steps; "
                  "prefill quantize-append of the sample took %.2f s (%.0f tokens/s)" % (
                      nb, wl.batch, wl.layers, wl.context, len(times), prefill_s, nb * wl.context / prefill_s),
        "append_prefill_tokens_per_s": nb * wl.context / prefill_s,
    }


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    leg = oracle_leg(wl, oracle_sequences(wl), args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": leg["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": leg["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, args.uniform_bits, args.scale_groups),
        "cpu_baseline": {"value": leg["value"], "unit": UNIT, "cores": leg["cores"], "kind": "oracle",
                         "sample": leg["sample"]},
        "e2e": {"value": leg["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


WORKLOAD_TEXT = {
    "cfg1": "SmolLM-135M-shaped single layer, 9 q / 3 kv heads, batch 1, context 512, bits iid {2:.40,4:.35,8:.20,16:.05}",
    "cfg2": "SmolLM-135M-shaped full cache, 30 layers, 9 q / 3 kv heads, batch 1, context 2048, controller bits",
    "cfg3": "SmolLM-360M-shaped, 32 layers, 15 q / 5 kv heads, batch 8, context 4096, controller bits",
    "cfg4": "SmolLM-1.7B-shaped, 24 layers, 32 q / 32 kv heads, batch 16, context 8192, bits in geometric runs "
            "{2:.25,4:.40,8:.25,16:.10} (or uniform with --uniform-bits)",
    "cfg5": "stress: 1 SmolLM-1.7B-shaped layer, 32 q / 32 kv heads, batch 16, context 32768, bits iid "
            "{2:.50,4:.30,8:.15,16:.05} seed 0",
}


def flushes_l2(wl) -> bool:
    """Small workloads would sit in the 126 MB L2 between steps: their timed steps run with L2 flushed.  Decided
    from the workload's shape alone (the fp16-equivalent size of its whole cache), so that every arm of the
    benchmark describes the same configuration."""
    return wl.layers * wl.batch * wl.kv_heads * wl.context * 256 < 2 * L2_BYTES


def workload_config(wl, uniform_bits=0, scale_groups=1):
    """The `config` object: a function of the workload definition only (identical in both arms)."""
    base = wl.name.split("-")[0]
    cfg = {"workload": "%s: %s; head_dim 64; each step appends 1 controller-decided token per sequence to every "
                       "layer and attends (this run: batch %d, context %d)" % (
                           wl.name, WORKLOAD_TEXT.get(base, base), wl.batch, wl.context),
           "layers": wl.layers, "batch": wl.batch, "q_heads": wl.q_heads, "kv_heads": wl.kv_heads,
           "head_dim": wl.head_dim, "context": wl.context}
    if flushes_l2(wl):
        cfg["l2"] = ("L2 flushed between timed steps (a 256 MB buffer is overwritten outside the timed region): "
                     "the whole cache is smaller than twice the 126 MB L2")
    else:
        cfg["l2"] = "inputs larger than L2: every step streams the packed KV of all layers, several times the 126 MB L2"
    if wl.bits_mode == "controller" or base == "cfg5":
        cfg["controller"] = ("MLP 4-%d-%d-4, Kaiming-uniform weights, seed %d (a seed for which all four classes "
                             "occur on the synthetic features)" % (wl.hidden, wl.hidden, wl.mlp_seed))
    if uniform_bits:
        cfg["uniform_bits"] = uniform_bits
    if scale_groups != 1:
        cfg["scale_groups"] = scale_groups
    return cfg


class Bench:
    """One process's device, library and process group."""

    def __init__(self):
        import torch
        from paper_2604_04722_b200 import binding as kq
        from paper_2604_04722_b200 import build as kbuild
        self.torch, self.kq = torch, kq
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=self.dev)
            self.dist = dist
        if self.rank == 0:
            kbuild.build()
        self.barrier()
        self.clib = kq.lib()
        self.stream = torch.cuda.current_stream().cuda_stream
        self.flush_buf = None
        self.kv_cache = {}                                  # host K/V blocks shared by the variants of a workload

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def to_dev(self, a, dt):
        return self.torch.from_numpy(np.ascontiguousarray(a).view(dt)).to(self.dev)

    def flush_l2(self, tag):
        if self.flush_buf is None:
            self.flush_buf = self.torch.empty(256 << 20, dtype=self.torch.uint8, device=self.dev)
        self.flush_buf.fill_(tag & 0xff)

    def timed_block(self, fn, reps):
        """Device time of `reps` calls of fn, bracketed by barrier + synchronize on both sides (ms)."""
        torch = self.torch
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(reps):
            fn()
        ev1.record()
        torch.cuda.synchronize()
        self.barrier()
        return ev0.elapsed_time(ev1)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def near_tie_report(bench, ctx, feats_d, n, max_rows=5):
    """Decisions whose two largest controller logits lie within NEAR_TIE_GAP of each other (Eq. 22-23), from
    the logits kvq_select_bits returns: count and the first few (token index, logits, gap, decision)."""
    torch, kq = bench.torch, bench.kq
    bits = torch.zeros(n, dtype=torch.uint8, device=bench.dev)
    logits = torch.zeros((n, 4), dtype=torch.float32, device=bench.dev)
    kq.kvq_select_bits(ctx, feats_d, n, bits, logits)
    top = torch.topk(logits, 2, dim=1).values
    gap = top[:, 0] - top[:, 1]
    idx = torch.nonzero(gap < NEAR_TIE_GAP).flatten()
    rows = [{"token": int(i), "logits": [float(x) for x in logits[i].tolist()], "gap": float(gap[i]),
             "bits": int(bits[i])} for i in idx[:max_rows].tolist()]
    return {"threshold": NEAR_TIE_GAP, "decisions": int(n), "count": int(idx.numel()), "first": rows}


def measure(bench, wl, *, steps, warmup, blocks, uniform_bits=0, scale_groups=1, e2e=True, e2e_blocks=3, k_per_channel=False):
    """Build the cache of `wl`, time its prefill, its decode steps and (optionally) the host-buffer steps."""
    torch, kq, dev, clib, stream = bench.torch, bench.kq, bench.dev, bench.clib, bench.stream
    W, K_steps = warmup, steps
    cold = flushes_l2(wl)
    e2e_warm = 3
    n_e2e = (e2e_warm + e2e_blocks * K_steps) if e2e else 0
    total_steps = W + blocks * K_steps + 2 * K_steps + n_e2e + 1
    L, B, Hq, Hkv, D, ctx_len = wl.layers, wl.batch, wl.q_heads, wl.kv_heads, wl.head_dim, wl.context
    seed = wl.seed + 1000 * bench.rank                # replicas draw their own data
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)

    # Every layer is filled with the same seeded K/V block (layer 0's): drawing 24 layers of cfg4 on the
    # host would take minutes and changes nothing the kernels see.
    t_gen = time.perf_counter()
    key = (seed, B, ctx_len, Hkv)
    if key not in bench.kv_cache:
        bench.kv_cache.clear()
        bench.kv_cache[key] = synth.kv_batch(seed, 0, B, 0, ctx_len, Hkv) + (synth.features_batch(seed, B, 0, ctx_len),)
    K, V, feats_prefill = bench.kv_cache[key]
    if uniform_bits:
        bits = np.full((B, ctx_len), uniform_bits, np.uint8)
    elif wl.bits_mode == "controller":
        bits = None                                   # decided on the device from the features
    else:
        wl_seeded = dataclasses.replace(wl, seed=seed)
        bits = np.stack([synth.workload_bits(wl_seeded, b, 0, ctx_len) for b in range(B)])
    t_gen = time.perf_counter() - t_gen

    to_dev = bench.to_dev
    if k_per_channel:
        ctx = kq.kvq_create_perchannel(L, Hq, Hkv, D, ctx_len + total_steps, B)
    elif scale_groups == 1:
        ctx = kq.kvq_create(L, Hq, Hkv, D, ctx_len + total_steps, B)
    else:
        ctx = kq.kvq_create_grouped(L, Hq, Hkv, D, ctx_len + total_steps, B, 0, scale_groups)
    kq.kvq_set_controller(ctx, cw.hidden, *cw.as_tuple())
    Kd, Vd = to_dev(K, np.int16), to_dev(V, np.int16)
    feats_d = to_dev(feats_prefill, np.float32)
    bits_d = to_dev(bits, np.uint8) if bits is not None else None

    def timed(fn, reps):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(reps):
            fn()
        ev1.record()
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1) / reps

    # ---- prefill quantize-append of one layer, timed both ways (kvq_reset empties every layer)
    ctl_bits = torch.zeros((B, ctx_len), dtype=torch.uint8, device=dev)

    def prefill_fused():
        kq.kvq_reset(ctx)
        kq.kvq_append_fused(ctx, 0, Kd, Vd, feats_d, ctx_len, ctl_bits)

    prefill_fused()
    ms_prefill_fused = timed(prefill_fused, 3)
    ctl_hist = {int(b): int((ctl_bits == b).sum().item()) for b in (2, 4, 8, 16)}
    ctl_written = sum(ROW_BYTES[b] * n for b, n in ctl_hist.items()) * Hkv
    near = near_tie_report(bench, ctx, feats_d, B * ctx_len)

    def prefill_same_bits():                          # the controller's own decisions, given: the same bytes are written
        kq.kvq_reset(ctx)
        kq.kvq_append(ctx, 0, Kd, Vd, ctl_bits, ctx_len)

    ms_prefill_same = timed(prefill_same_bits, 3)
    if bits_d is None:                                # controller workloads keep the controller's decisions
        bits_d = ctl_bits
        bits = ctl_bits.cpu().numpy()

    def prefill_given():
        kq.kvq_reset(ctx)
        kq.kvq_append(ctx, 0, Kd, Vd, bits_d, ctx_len)

    ms_prefill_given = timed(prefill_given, 3)
    given_hist = {int(b): int((bits == b).sum()) for b in (2, 4, 8, 16)}
    given_written = sum(ROW_BYTES[b] * n for b, n in given_hist.items()) * Hkv
    for layer in range(1, L):                         # the other layers get the same tokens (untimed)
        kq.kvq_append(ctx, layer, Kd, Vd, bits_d, ctx_len)
    torch.cuda.synchronize()
    del Kd, Vd, feats_d
    torch.cuda.empty_cache()

    # ---- per-step inputs, resident on the device (shared by the layers); one draw per sequence
    f_steps = np.stack([synth.features(seed, b, ctx_len, total_steps) for b in range(B)], axis=1)[:, :, None, :]   # [S][B][1][4]
    kv_steps = [synth.kv_rows(seed, 0, b, ctx_len, total_steps, Hkv) for b in range(B)]
    k_steps = np.ascontiguousarray(np.stack([kv[0] for kv in kv_steps], axis=1)[:, :, None])     # [S][B][1][Hkv][64]
    v_steps = np.ascontiguousarray(np.stack([kv[1] for kv in kv_steps], axis=1)[:, :, None])
    q_rng = np.random.default_rng([seed & 0xffffffff, 77, ctx_len])
    q_steps = q_rng.standard_normal((total_steps, B, Hq, D), dtype=np.float32).astype(np.float16)
    f_steps = np.ascontiguousarray(f_steps)
    f_d, k_d, v_d, q_d = to_dev(f_steps, np.float32), to_dev(k_steps, np.int16), to_dev(v_steps, np.int16), \
        to_dev(q_steps, np.int16)
    O_d = torch.zeros((B, Hq, D), dtype=torch.int16, device=dev)
    step_bits_d = torch.zeros((total_steps, B), dtype=torch.uint8, device=dev)

    step_no = [0]

    # The timed loop passes plain addresses to the C calls: slicing tensors and re-deriving their pointers
    # costs more host time per call than a small workload's kernels take.
    ptr = lambda t: [t[i].data_ptr() for i in range(t.shape[0])]
    k_p, v_p, f_p, q_p, sb_p = ptr(k_d), ptr(v_d), ptr(f_d), ptr(q_d), ptr(step_bits_d)
    O_p = O_d.data_ptr()

    def one_step():
        s = step_no[0]
        for layer in range(L):
            rc = clib.kvq_decode_step(ctx, layer, f_p[s], k_p[s], v_p[s], q_p[s], O_p, sb_p[s], stream)
            if rc:
                raise kq.KvqError(rc, "decode step")
        step_no[0] = s + 1

    for _ in range(W):
        one_step()
    torch.cuda.synchronize()
    _, resident0, _ = kq.kvq_stats(ctx, 0, B)

    sampler = ClockSampler(bench.local)
    sampler.start()
    time.sleep(0.25)
    launches1 = kq.kvq_launch_count(ctx)
    attn_ms, ncalls = 0.0, 0
    block_ms, warm_ms = [], None
    launches_block = None
    if cold:
        # one pair of events per step; the flush runs between the pairs, outside the timed regions
        for _ in range(blocks):
            ms_total = 0.0
            for _ in range(K_steps):
                bench.flush_l2(step_no[0])
                ms_total += bench.timed_block(one_step, 1)
            block_ms.append(ms_total)
            if launches_block is None:
                launches_block = kq.kvq_launch_count(ctx) - launches1
        # one more block with the library's event pair around every launch (the pairs keep the launches of
        # neighbouring layers from overlapping, so the steps above are timed without them)
        kq.kvq_set_profiling(ctx, True)
        kq.kvq_profile_read(ctx)
        for _ in range(K_steps):
            bench.flush_l2(step_no[0])
            bench.timed_block(one_step, 1)
            a_ms, n = kq.kvq_profile_read(ctx)
            attn_ms, ncalls = attn_ms + a_ms, ncalls + n
        kq.kvq_set_profiling(ctx, False)
        warm_ms = bench.timed_block(one_step, K_steps)         # the same steps with whatever stays in L2
    else:
        for _ in range(blocks):
            block_ms.append(bench.timed_block(one_step, K_steps))
            if launches_block is None:
                launches_block = kq.kvq_launch_count(ctx) - launches1
        # The attention kernel's own duration: one more block, now with the library's event pair around
        # every attention launch.  The events sit between the append and the attention kernel and keep
        # the two from overlapping, so this pass is not the one `value` is taken from.
        kq.kvq_set_profiling(ctx, True)
        kq.kvq_profile_read(ctx)
        ms_instrumented = bench.timed_block(one_step, K_steps)
        attn_ms, ncalls = kq.kvq_profile_read(ctx)
        kq.kvq_set_profiling(ctx, False)
    time.sleep(0.1)
    clocks = sampler.stop()
    steps_done = step_no[0]
    _, resident1, ebits = kq.kvq_stats(ctx, 0, B)
    arena_used, arena_total, arena_block = kq.kvq_arena_usage(ctx)
    resident_mean = 0.5 * (resident0 + resident1)     # per layer
    new_rows_mean = (resident1 - resident0) / max(1, steps_done - W)
    flags = kq.kvq_device_status(ctx)

    # ---- end to end through the host-buffer entry point (pinned buffers, copies timed)
    e2e_ms = []
    if e2e:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        f_h, k_h, v_h, q_h = pin(f_steps.view(np.float32)), pin(k_steps.view(np.int16)), pin(v_steps.view(np.int16)), \
            pin(q_steps.view(np.int16))
        O_h = torch.zeros((B, Hq, D), dtype=torch.int16).pin_memory()
        fh_p, kh_p, vh_p, qh_p, Oh_p = ptr(f_h), ptr(k_h), ptr(v_h), ptr(q_h), O_h.data_ptr()

        def one_step_host():
            s = step_no[0]
            for layer in range(L):
                rc = clib.kvq_decode_step_host(ctx, layer, fh_p[s], kh_p[s], vh_p[s], qh_p[s], Oh_p, None, stream)
                if rc:
                    raise kq.KvqError(rc, "decode step from host buffers")
            step_no[0] = s + 1

        for _ in range(e2e_warm):
            one_step_host()
        for _ in range(e2e_blocks):
            if cold:
                ms_total = 0.0
                for _ in range(K_steps):
                    bench.flush_l2(step_no[0])
                    ms_total += bench.timed_block(one_step_host, 1)
                e2e_ms.append(ms_total)
            else:
                e2e_ms.append(bench.timed_block(one_step_host, K_steps))
    h2d = L * (B * 16 + 2 * B * Hkv * D * 2 + B * Hq * D * 2)
    d2h = L * B * Hq * D * 2

    # ---- reduce over ranks: slowest rank's time for every block, summed bytes
    dec_bytes, app_bytes = step_bytes(wl, resident_mean, new_rows_mean)            # per layer, this rank's replica
    ms_attn = attn_ms / max(ncalls, 1)
    per_step = [t / K_steps for t in block_ms]
    e2e_per_step = [t / K_steps for t in e2e_ms]
    reduced, bytes_job = aggregate_over_ranks(per_step + e2e_per_step + [ms_attn], L * (dec_bytes + app_bytes),
                                              bench.dist, dev)
    per_step, e2e_per_step, ms_attn = reduced[:len(per_step)], reduced[len(per_step):-1], reduced[-1]
    ms_step = float(np.median(per_step))
    ms_e2e = float(np.median(e2e_per_step)) if e2e_per_step else None
    peak, peak_kind = measured_peak_gbs()
    # The kernel the roofline is quoted on.  When a step is ONE kernel per layer (k_decode_step), its average launch
    # duration is the timed region itself divided by the launches in it (K * L back-to-back launches between one pair
    # of events) and its algorithmic bytes are the whole step's; the library's event pair around every single launch
    # (which keeps neighbouring launches from overlapping) is reported beside it.  With two kernels per layer the
    # attention kernel is timed by those event pairs.
    one_kernel = int(launches_block) == K_steps * L
    ms_launch = ms_step / L if one_kernel else ms_attn
    launch_bytes = dec_bytes + app_bytes if one_kernel else dec_bytes
    achieved = launch_bytes / (ms_launch * 1e-3) / 1e9
    index_bytes = B * (ctx_len + 0.5 * (W + steps_done)) * 4
    kq.kvq_destroy(ctx)
    del f_d, k_d, v_d, q_d, O_d, step_bits_d
    torch.cuda.empty_cache()
    return {
        "ms_step": ms_step, "ms_step_min": float(min(per_step)), "ms_step_max": float(max(per_step)),
        "ms_step_blocks": per_step, "ms_e2e": ms_e2e, "ms_e2e_blocks": e2e_per_step, "ms_attn": ms_attn,
        "ms_warm": None if warm_ms is None else warm_ms / K_steps,
        "ms_instrumented": None if cold else ms_instrumented / K_steps,
        "bytes_job": bytes_job, "dec_bytes": dec_bytes, "app_bytes": app_bytes, "achieved": achieved, "peak": peak,
        "ms_launch": ms_launch, "launch_bytes": launch_bytes,
        "peak_kind": peak_kind, "index_bytes": index_bytes, "clocks": clocks, "cold": cold, "h2d": h2d, "d2h": d2h,
        "launches_block": int(launches_block), "device_flags": int(flags), "near_ties": near,
        # kvq_decode_step runs one kernel per layer on short caches (k_decode_step: the attending warps add the
        # step's token themselves), two otherwise; the library's event pair is around the attending kernel
        "step_kernels": ("k_decode_step" if int(launches_block) == K_steps * L else "k_append_token + k_decode_attn"),
        "prefill": {
            "controller_fused": B * ctx_len / (ms_prefill_fused * 1e-3),
            "bits_given": B * ctx_len / (ms_prefill_given * 1e-3),
            "ms_fused": ms_prefill_fused, "ms_bits_given": ms_prefill_given,
            "ms_bits_given_same_bits_as_fused": ms_prefill_same,
            "GBps_fused": (B * ctx_len * Hkv * 256 + ctl_written) / (ms_prefill_fused * 1e-3) / 1e9,
            "GBps_bits_given": (B * ctx_len * Hkv * 256 + given_written) / (ms_prefill_given * 1e-3) / 1e9,
            "frac_of_peak_bits_given": (B * ctx_len * Hkv * 256 + given_written) / (ms_prefill_given * 1e-3) / 1e9 / peak,
            "controller_class_histogram": ctl_hist, "note": "one layer"},
        "memory": {"packed_row_bytes": int(L * resident1), "arena_bytes_in_use": int(arena_used * arena_block),
                   "arena_bytes_reserved": int(arena_total * arena_block),
                   "fp16_cache_bytes": int(L * B * Hkv * (ctx_len + steps_done) * 256),
                   "note": "arena blocks are taken on demand; kvq_create reserves the worst case, "
                           "kvq_create_arena any budget"},
        "expected_bits": ebits, "input_generation_s": t_gen, "steps_run": steps_done,
    }


def compact(m, wl, cpu=None):
    """The short form of a measurement for `other_workloads`."""
    out = {
        "config": {"layers": wl.layers, "batch": wl.batch, "q_heads": wl.q_heads, "kv_heads": wl.kv_heads, "context": wl.context,
                   "l2": "flushed between steps" if m["cold"] else "inputs larger than L2"},
        "step_us": m["ms_step"] * 1e3, "step_us_min": m["ms_step_min"] * 1e3, "step_us_max": m["ms_step_max"] * 1e3,
        "step_us_warm_l2": None if m["ms_warm"] is None else m["ms_warm"] * 1e3,
        "decode_attn_us_per_layer": m["ms_attn"] * 1e3, "step_kernels_per_layer": m["step_kernels"],
        "roofline_kernel_us_per_launch": m["ms_launch"] * 1e3,
        "kv_bytes_per_layer": m["dec_bytes"], "decode_GBps": m["achieved"], "frac_of_measured_hbm": m["achieved"] / m["peak"],
        "value_GBps": m["bytes_job"] / (m["ms_step"] * 1e-3) / 1e9,
        "prefill_ms_fused": m["prefill"]["ms_fused"], "prefill_ms_bits_given": m["prefill"]["ms_bits_given"],
        "prefill_tokens_per_s_fused": m["prefill"]["controller_fused"],
        "prefill_tokens_per_s_bits_given": m["prefill"]["bits_given"],
        "controller_class_histogram": m["prefill"]["controller_class_histogram"],
        "near_ties": {"count": m["near_ties"]["count"], "decisions": m["near_ties"]["decisions"]},
        "clocks": {k: m["clocks"].get(k) for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples")},
        "gpu_launches_per_block": m["launches_block"], "device_flags": m["device_flags"],
    }
    if cpu is not None:
        out["cpu_baseline"] = cpu
    return out


def cpu_leg(wl, steps, warmup=1):
    leg = oracle_leg(wl, oracle_sequences(wl), steps, warmup)
    return {"value": leg["value"], "unit": UNIT, "cores": leg["cores"], "kind": "oracle", "sample": leg["sample"],
            "ms_per_step_of_sample": leg["ms_per_step"],
            "append_prefill_tokens_per_s": leg["append_prefill_tokens_per_s"]}


def measure_feature_kernels(bench, n=4096, vocab=49152, reps=5):
    """The on-device feature kernel (Eq. 14-17: entropy, rarity, confidence of n tokens from their logits):
    one pass over the logits, so its bound is HBM.  Synthetic logits (the kernel's time does not depend on
    their values), larger than L2 in both types."""
    torch, kq = bench.torch, bench.kq
    peak, _ = measured_peak_gbs()
    out = {"tokens": n, "vocab": vocab, "note": "kvq_token_features, one launch, logits resident in HBM; bytes = the logits"}
    ids = torch.randint(0, vocab, (n,), dtype=torch.int32, device=bench.dev)
    counts = torch.randint(0, 5000, (vocab,), dtype=torch.int32, device=bench.dev)
    feats = torch.zeros((n, 4), dtype=torch.float32, device=bench.dev)
    for name, dt in (("fp32", torch.float32), ("fp16", torch.float16)):
        logits = (torch.randn((n, vocab), device=bench.dev, dtype=torch.float32) * 3).to(dt)
        fn = lambda: kq.kvq_token_features(logits, dt == torch.float32, n, vocab, ids, counts, 10_000_000, vocab // 2, None, feats)
        fn()
        ms = bench.timed_block(fn, reps) / reps
        nbytes = logits.numel() * logits.element_size()
        out[name] = {"us_per_launch": ms * 1e3, "GBps": nbytes / (ms * 1e-3) / 1e9, "frac_of_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / peak,
                     "logit_bytes": nbytes}
        del logits
    torch.cuda.empty_cache()
    return out


def run_ours(args, wl):
    bench = Bench()
    rank, world = bench.rank, bench.world
    is_headline = wl.name == "cfg5" and not args.uniform_bits and args.scale_groups == 1 and not args.k_per_channel
    m = measure(bench, wl, steps=args.steps, warmup=args.warmup, blocks=args.blocks, uniform_bits=args.uniform_bits,
                scale_groups=args.scale_groups, k_per_channel=args.k_per_channel)

    others = None
    if is_headline and world == 1 and not args.no_other_workloads:
        others = {}
        for name, ub in (("cfg1", 0), ("cfg2", 0), ("cfg3", 0), ("cfg4", 0), ("cfg4", 2), ("cfg4", 4), ("cfg4", 8), ("cfg4", 16)):
            w2 = synth.CONFIGS[name]
            m2 = measure(bench, w2, steps=args.other_steps, warmup=3, blocks=args.other_blocks, uniform_bits=ub, e2e=False)
            cpu2 = None
            if not args.no_cpu_baseline and not ub:
                cpu2 = cpu_leg(w2, 3)
            others[name + ("_all_%d_bit" % ub if ub else "")] = compact(m2, w2, cpu2)
        bench.kv_cache.clear()
    features = measure_feature_kernels(bench) if is_headline and world == 1 and not args.no_other_workloads else None

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and is_headline:
        cpu = cpu_leg(wl, 20)

    if rank == 0:
        traffic, traffic_note = (recorded_traffic() if is_headline and wl.batch == 16 and wl.context == 32768
                                 else (None, "not the captured workload"))
        ms_step, ms_e2e, ms_attn = m["ms_step"], m["ms_e2e"], m["ms_attn"]
        sm = m["clocks"].get("sm_mhz")
        line = {
            "metric": METRIC, "value": m["bytes_job"] / (ms_step * 1e-3) / 1e9, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(wl, args.uniform_bits, args.scale_groups), **({"k_per_channel": True} if args.k_per_channel else {})),
            "timing": {"blocks": args.blocks, "steps_per_block": args.steps,
                       "ms_per_step_median": ms_step, "ms_per_step_min": m["ms_step_min"], "ms_per_step_max": m["ms_step_max"],
                       "ms_per_step_of_each_block": m["ms_step_blocks"],
                       "ms_per_step_x_sm_mhz": None if sm is None else ms_step * sm,
                       "note": "each block is exactly `steps` steps between device synchronisations; median block reported"},
            "clocks": m["clocks"],
            "e2e": {"value": m["bytes_job"] / (ms_e2e * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms_e2e,
                    "ms_per_step_of_each_block": m["ms_e2e_blocks"],
                    "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"]},
            "gpu_launches": m["launches_block"],
            "roofline": {"bound": "hbm", "kernel": "k_decode_step" if m["step_kernels"] == "k_decode_step" else "k_decode_attn", "achieved": m["achieved"], "peak": m["peak"],
                         "unit": "GB/s", "frac": m["achieved"] / m["peak"], "peak_kind": "of " + m["peak_kind"],
                         "traffic": traffic, "traffic_note": traffic_note,
                         "algorithmic_bytes_per_launch": m["launch_bytes"],
                         "avg_launch_us": m["ms_launch"] * 1e3,
                         "avg_launch_us_event_pair_per_launch": ms_attn * 1e3,
                         "timed_in": ("the timed blocks: steps x layers back-to-back launches of the step kernel between one pair of "
                                      "events; the event-pair figure is from the library's events around every single launch"
                                      if m["step_kernels"] == "k_decode_step" else
                                      "one more block of steps (L2 flushed before each), one event pair per launch" if m["cold"] else
                                      "one more block of the same number of steps with an event pair around every launch"),
                         "frac_with_index_bytes": (m["launch_bytes"] + m["index_bytes"]) / (m["ms_launch"] * 1e-3) / 1e9 / m["peak"]},
            "cpu_baseline": cpu,
            "decode_attn_us_per_layer": ms_attn * 1e3, "step_kernels_per_layer": m["step_kernels"],
            "step_us": ms_step * 1e3,
            "step_us_warm_l2": None if m["ms_warm"] is None else m["ms_warm"] * 1e3,
            "step_us_with_kernel_events": None if m["ms_instrumented"] is None else m["ms_instrumented"] * 1e3,
            "append_prefill_tokens_per_s": m["prefill"],
            "near_ties": m["near_ties"],
            "memory": m["memory"],
            "kv_bytes_per_layer": m["dec_bytes"], "expected_bits": m["expected_bits"],
            "device_flags": m["device_flags"], "input_generation_s": m["input_generation_s"],
            "other_workloads": others,
            "feature_kernels": features,
        }
        print(json.dumps(line))
    bench.close()


SWEEP_SPLITS = (1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 12, 14, 16, 18, 20, 24, 28, 32, 40, 48, 56, 64)


def run_sweep(args):
    """The automatic launch plan of kvq_decode_attn against every explicit split count, per workload (one layer
    of each; L2 flushed before every launch of the small ones).  Prints one JSON line; not a benchmark result."""
    bench = Bench()
    torch, kq, dev = bench.torch, bench.kq, bench.dev
    out = {}
    for name, ub in (("cfg1", 0), ("cfg2", 0), ("cfg3", 0), ("cfg4", 0), ("cfg4", 2), ("cfg4", 16), ("cfg5", 0)):
        wl = synth.CONFIGS[name]
        B, Hq, Hkv, n = wl.batch, wl.q_heads, wl.kv_heads, wl.context
        K, V = synth.kv_batch(wl.seed, 0, B, 0, n, Hkv)
        cw = synth.controller_weights(wl.mlp_seed, wl.hidden)
        ctx = kq.kvq_create(1, Hq, Hkv, 64, n, B)
        kq.kvq_set_controller(ctx, cw.hidden, *cw.as_tuple())
        Kd, Vd = bench.to_dev(K, np.int16), bench.to_dev(V, np.int16)
        if ub:
            kq.kvq_append(ctx, 0, Kd, Vd, bench.to_dev(np.full((B, n), ub, np.uint8), np.uint8), n)
        elif wl.bits_mode == "controller":
            kq.kvq_append_fused(ctx, 0, Kd, Vd, bench.to_dev(synth.features_batch(wl.seed, B, 0, n), np.float32), n, None)
        else:
            kq.kvq_append(ctx, 0, Kd, Vd, bench.to_dev(np.stack([synth.workload_bits(wl, b, 0, n) for b in range(B)]), np.uint8), n)
        del Kd, Vd
        Qd = bench.to_dev(synth.queries(wl.seed, 0, 0, B, Hq), np.int16)
        O = torch.zeros_like(Qd)
        cold = flushes_l2(dataclasses.replace(wl, layers=1))
        reps = 30 if cold else 10

        def time_plan(splits):
            kq.kvq_set_splits(ctx, splits)
            kq.kvq_decode_attn(ctx, 0, Qd, O)
            ts = []
            for r in range(reps):
                if cold:
                    bench.flush_l2(r)
                ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                ev0.record()
                kq.kvq_decode_attn(ctx, 0, Qd, O)
                ev1.record()
                torch.cuda.synchronize()
                ts.append(ev0.elapsed_time(ev1) * 1e3)
            return float(np.median(ts))

        auto = time_plan(0)
        explicit = {s: time_plan(s) for s in SWEEP_SPLITS}
        best = min(explicit, key=explicit.get)
        out[name + ("_all_%d_bit" % ub if ub else "")] = {
            "automatic_us": auto, "best_explicit_splits": best, "best_explicit_us": explicit[best],
            "automatic_over_best": auto / explicit[best], "explicit_us": explicit, "l2": "flushed" if cold else "larger than L2"}
        kq.kvq_destroy(ctx)
        torch.cuda.empty_cache()
    print(json.dumps({"sweep_splits": out, "note": "median of %s launches per plan, CUDA events around the attention launch only"
                      % "10-30"}))
    bench.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100, help="steps per timed block")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--blocks", type=int, default=10, help="timed blocks of `--steps` steps; the median is reported")
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing legs")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the other workloads that the default line carries beside the headline one")
    ap.add_argument("--other-steps", type=int, default=10, help="steps per block of the other workloads")
    ap.add_argument("--other-blocks", type=int, default=5)
    ap.add_argument("--features-only", action="store_true",
                    help="time only the on-device feature kernel (the `feature_kernels` object of the default line)")
    ap.add_argument("--sweep-splits", action="store_true",
                    help="compare the automatic launch plan of the attention kernel with explicit split counts")
    ap.add_argument("--context", type=int, default=0,
                    help="shorter cached context than the workload's 32768, for profiler captures that must "
                         "stay small; the printed config names it and the line is not a benchmark result")
    ap.add_argument("--workload", choices=sorted(synth.CONFIGS), default="cfg5",
                    help="cfg5 (default) is the workload the metric is quoted on; cfg1..cfg4 are the other SmolLM-shaped workloads")
    ap.add_argument("--uniform-bits", type=int, choices=[2, 4, 8, 16], default=0,
                    help="store every prefill token at this precision (the static baselines of cfg4)")
    ap.add_argument("--scale-groups", type=int, choices=[1, 2], default=1,
                    help="2: one scale / zero-point pair per 32 channels instead of per row (a variant, not the "
                         "quantizer the metric is quoted on)")
    ap.add_argument("--k-per-channel", action="store_true",
                    help="keys quantized per channel over windows of 16 slots (a variant, not the quantizer the metric is quoted on)")
    ap.add_argument("--batch", type=int, default=0,
                    help="fewer sequences than the workload's 16, likewise for profiler captures only")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    args.blocks = max(1, args.blocks)
    wl = synth.CONFIGS[args.workload]
    if args.context > 0:
        wl = dataclasses.replace(wl, context=args.context, name="%s-context-%d" % (wl.name, args.context))
    if args.batch > 0:
        wl = dataclasses.replace(wl, batch=args.batch, name="%s-batch-%d" % (wl.name, args.batch))
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.sweep_splits:
        run_sweep(args)
    elif args.features_only:
        b = Bench()
        if b.rank == 0:
            print(json.dumps({"feature_kernels": measure_feature_kernels(b)}))
        b.close()
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
