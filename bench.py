#!/usr/bin/env python
"""Benchmark of the adaptive KV-cache hot path on B200.

A "step" is one pass of the whole path over one batch of synthetic input: controller decision
for the step's new tokens (Eq. 19-23), quantize-append of their K/V rows (Eq. 24, Eq. 4) and
decode attention over the whole mixed-precision cache (Eq. 5).  The workload is the stress
configuration the bandwidth target is quoted on: one SmolLM-1.7B-shaped layer, 32 query / 32 KV
heads, head_dim 64, batch 16, context 32768, bit-widths i.i.d. {2:50%, 4:30%, 8:15%, FP16:5%}.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference ...                     # the CPU oracle on a bounded sample

With N > 1 (launched by torchrun) every rank runs an independent replica of the workload (the
path has no exchange step); the reported value is the sum over ranks divided by the slowest
rank's device time.

Prints ONE JSON line.  `value` = algorithmic bytes of a step (packed codes + scales read by the
attention, Q/O, the new tokens' fp16 rows read and packed rows + index written, their features)
per second, inputs resident in HBM.  `e2e` = the same through kvq_decode_step_host with pinned
host buffers, copies inside the timed region.
"""
from __future__ import annotations

import argparse
import dataclasses
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

# DRAM traffic of one k_decode_attn launch on this workload (dram__bytes_read.sum +
# dram__bytes_write.sum): captured with a quarter of the sequences (profiles/k_decode_attn_cfg5_batch4.md,
# 320.0 MB per launch) and scaled by the rows read (x 4); every row is read exactly once, so traffic
# grows in proportion.  Set to None whenever the kernel changes after the capture.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 4 * 320.0e6


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def step_bytes(wl, n_cached_mean, resident_bytes_mean, new_row_bytes_mean):
    """Algorithmic bytes of one step (per replica)."""
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
                 "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
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
        sm, smax, reasons = [], [], set()
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1]))
                    smax.append(float(p[2]))
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
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)), samples=len(sm))
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


def oracle_leg(wl, seqs, steps, warmup):
    """The CPU oracle, as it stands, on a bounded sample of the workload: `seqs` whole sequences.
    Each step = decision for the new tokens + quantize-append + attention over everything cached."""
    import oracle
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)
    nb = len(seqs)
    K = np.stack([synth.kv_rows(wl.seed, 0, b, 0, wl.context, wl.kv_heads)[0] for b in seqs])
    V = np.stack([synth.kv_rows(wl.seed, 0, b, 0, wl.context, wl.kv_heads)[1] for b in seqs])
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
        "sample": "%d of %d sequences of the workload (whole sequences, every head, one layer, context %d); %d steps; "
                  "prefill quantize-append of the sample took %.1f s (%.0f tokens/s)" % (
                      nb, wl.batch, wl.context, len(times), prefill_s, nb * wl.context / prefill_s),
        "append_prefill_tokens_per_s": nb * wl.context / prefill_s,
    }


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    leg = oracle_leg(wl, [0], args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": leg["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": leg["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl),
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


def workload_config(wl, cold=None, kv_bytes_all_layers=None):
    base = wl.name.split("-")[0]
    cfg = {"workload": "%s: %s; head_dim 64; each step appends 1 controller-decided token per sequence to every "
                       "layer and attends (this run: batch %d, context %d)" % (
                           wl.name, WORKLOAD_TEXT.get(base, base), wl.batch, wl.context),
           "layers": wl.layers, "batch": wl.batch, "q_heads": wl.q_heads, "kv_heads": wl.kv_heads,
           "head_dim": wl.head_dim, "context": wl.context}
    if cold is None:
        cfg["l2"] = "inputs larger than L2 (126 MB) for cfg4/cfg5; smaller workloads flush L2 between timed steps"
    elif cold:
        cfg["l2"] = ("L2 flushed between timed steps (a 256 MB buffer is overwritten outside the timed region): the "
                     "packed KV of all layers is %.1f MB, it would stay resident in the 126 MB L2" % (
                         kv_bytes_all_layers / 1e6))
    else:
        cfg["l2"] = "inputs larger than L2 (%.2f GB of packed KV is streamed per step; L2 is 126 MB)" % (
            kv_bytes_all_layers / 1e9)
    return cfg


def run_ours(args, wl):
    import torch
    from paper_2604_04722_b200 import binding as kq
    from paper_2604_04722_b200 import build as kbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        kbuild.build()
    if dist is not None:
        dist.barrier()
    kq.lib()

    W, K_steps = args.warmup, args.steps
    e2e_steps, e2e_warm = K_steps, max(3, W)
    total_steps = W + 2 * K_steps + e2e_warm + e2e_steps      # the flushed-L2 mode times its steps twice
    L, B, Hq, Hkv, D, ctx_len = wl.layers, wl.batch, wl.q_heads, wl.kv_heads, wl.head_dim, wl.context
    seed = wl.seed + 1000 * rank                      # replicas draw their own data
    cw = synth.controller_weights(wl.mlp_seed, wl.hidden)

    # Every layer is filled with the same seeded K/V block (layer 0's): drawing 24 layers of cfg4 on the
    # host would take minutes and changes nothing the kernels see.
    t_gen = time.perf_counter()
    K, V = synth.kv_batch(seed, 0, B, 0, ctx_len, Hkv)
    feats_prefill = synth.features_batch(seed, B, 0, ctx_len)
    if args.uniform_bits:
        bits = np.full((B, ctx_len), args.uniform_bits, np.uint8)
    elif wl.bits_mode == "controller":
        bits = None                                   # decided on the device from the features
    else:
        wl_seeded = dataclasses.replace(wl, seed=seed)
        bits = np.stack([synth.workload_bits(wl_seeded, b, 0, ctx_len) for b in range(B)])
    t_gen = time.perf_counter() - t_gen

    def to_dev(a, dt):
        return torch.from_numpy(np.ascontiguousarray(a).view(dt)).to(dev)

    if args.scale_groups == 1:
        ctx = kq.kvq_create(L, Hq, Hkv, D, ctx_len + total_steps, B)
    else:
        ctx = kq.kvq_create_grouped(L, Hq, Hkv, D, ctx_len + total_steps, B, 0, args.scale_groups)
    kq.kvq_set_controller(ctx, cw.hidden, *cw.as_tuple())
    Kd, Vd = to_dev(K, np.int16), to_dev(V, np.int16)
    feats_d = to_dev(feats_prefill, np.float32)
    bits_d = to_dev(bits, np.uint8) if bits is not None else None
    stream = torch.cuda.current_stream().cuda_stream

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
    launches0 = kq.kvq_launch_count(ctx)
    ctl_bits = torch.zeros((B, ctx_len), dtype=torch.uint8, device=dev)

    def prefill_fused():
        kq.kvq_reset(ctx)
        kq.kvq_append_fused(ctx, 0, Kd, Vd, feats_d, ctx_len, ctl_bits)

    prefill_fused()
    ms_prefill_fused = timed(prefill_fused, 3)
    ctl_hist = {int(b): int((ctl_bits == b).sum().item()) for b in (2, 4, 8, 16)}
    ctl_written = sum(ROW_BYTES[b] * n for b, n in ctl_hist.items()) * Hkv
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

    # ---- per-step inputs, resident on the device (shared by the layers)
    f_steps = np.stack([synth.features_batch(seed, B, ctx_len + s, 1) for s in range(total_steps)])   # [S][B][1][4]
    kv_steps = [synth.kv_batch(seed, 0, B, ctx_len + s, 1, Hkv) for s in range(total_steps)]
    k_steps = np.stack([kv[0] for kv in kv_steps])
    v_steps = np.stack([kv[1] for kv in kv_steps])
    q_steps = np.stack([synth.queries(seed, 0, s, B, Hq) for s in range(total_steps)])
    f_d, k_d, v_d, q_d = to_dev(f_steps, np.float32), to_dev(k_steps, np.int16), to_dev(v_steps, np.int16), \
        to_dev(q_steps, np.int16)
    O_d = torch.zeros((B, Hq, D), dtype=torch.int16, device=dev)
    step_bits_d = torch.zeros((total_steps, B), dtype=torch.uint8, device=dev)

    step_no = [0]

    # The timed loop passes plain addresses to the C calls: slicing tensors and re-deriving their pointers
    # costs more host time per call than a small workload's kernels take.
    clib = kq.lib()
    ptr = lambda t: [t[i].data_ptr() for i in range(t.shape[0])]
    k_p, v_p, f_p, q_p, sb_p = ptr(k_d), ptr(v_d), ptr(f_d), ptr(q_d), ptr(step_bits_d)
    O_p = O_d.data_ptr()

    def one_step():
        s = step_no[0]
        for layer in range(L):
            rc = clib.kvq_append_fused(ctx, layer, k_p[s], v_p[s], f_p[s], 1, sb_p[s], stream)
            rc = rc or clib.kvq_decode_attn(ctx, layer, q_p[s], O_p, stream)
            if rc:
                raise kq.KvqError(rc, "decode step")
        step_no[0] = s + 1

    _, resident_layer0, _ = kq.kvq_stats(ctx, 0, B)
    cold = L * resident_layer0 < 2 * 126e6            # the whole cache would sit in L2: flush it between steps
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if cold else None

    for _ in range(W):
        one_step()
    torch.cuda.synchronize()
    _, resident0, _ = kq.kvq_stats(ctx, 0, B)

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    if dist is not None:
        dist.barrier()
    launches1 = kq.kvq_launch_count(ctx)
    attn_ms, ncalls = 0.0, 0
    ms_instrumented = None
    if cold:
        # one pair of events per step; the flush runs between the pairs, outside the timed regions
        kq.kvq_set_profiling(ctx, True)
        kq.kvq_profile_read(ctx)
        ms_total = 0.0
        for _ in range(K_steps):
            flush_buf.fill_(step_no[0] & 0xff)
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            ev0.record()
            one_step()
            ev1.record()
            torch.cuda.synchronize()
            ms_total += ev0.elapsed_time(ev1)
            a_ms, n = kq.kvq_profile_read(ctx)
            attn_ms, ncalls = attn_ms + a_ms, ncalls + n
        ms_warm = timed(one_step, K_steps)            # the same steps again with whatever stays in L2
        kq.kvq_profile_read(ctx)
    else:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(K_steps):
            one_step()
        ev1.record()
        torch.cuda.synchronize()
        ms_total = ev0.elapsed_time(ev1)
        launches2 = kq.kvq_launch_count(ctx)
        # The attention kernel's own duration: the same number of steps once more, now with the library's
        # event pair around every attention launch.  The events sit between the append and the attention
        # kernel and keep the two from overlapping, so this pass is not the one `value` is taken from.
        kq.kvq_set_profiling(ctx, True)
        kq.kvq_profile_read(ctx)
        ms_instrumented = timed(one_step, K_steps)
        attn_ms, ncalls = kq.kvq_profile_read(ctx)
        ms_warm = None
    if dist is not None:
        dist.barrier()
    launches_timed = (kq.kvq_launch_count(ctx) - launches1) // 2 if cold else launches2 - launches1
    kq.kvq_set_profiling(ctx, False)
    time.sleep(0.2)
    clocks = sampler.stop()
    _, resident1, ebits = kq.kvq_stats(ctx, 0, B)
    arena_used, arena_total, arena_block = kq.kvq_arena_usage(ctx)
    resident_mean = 0.5 * (resident0 + resident1)     # per layer
    new_rows_mean = (resident1 - resident0) / max(1, step_no[0] - W)

    # ---- end to end through the host-buffer entry point (pinned buffers, copies timed)
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
    if dist is not None:
        dist.barrier()
    ms_e2e = timed(one_step_host, e2e_steps)
    if dist is not None:
        dist.barrier()
    h2d = L * (B * 16 + 2 * B * Hkv * D * 2 + B * Hq * D * 2)
    d2h = L * B * Hq * D * 2

    # ---- reduce over ranks: slowest rank's time, summed bytes
    ms_step = ms_total / K_steps
    dec_bytes, app_bytes = step_bytes(wl, ctx_len, resident_mean, new_rows_mean)    # per layer, this rank's replica
    (ms_step, ms_e2e, ms_attn), bytes_job = aggregate_over_ranks(
        [ms_step, ms_e2e, attn_ms / max(ncalls, 1)], L * (dec_bytes + app_bytes), dist, dev)
    peak, peak_kind = measured_peak_gbs()
    achieved = dec_bytes / (ms_attn * 1e-3) / 1e9
    index_bytes = B * (ctx_len + W + K_steps / 2) * 4
    is_headline = wl.name == "cfg5" and not args.uniform_bits and args.scale_groups == 1

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and is_headline:
        leg = oracle_leg(wl, [0, 1], 20, 1)
        cpu = {"value": leg["value"], "unit": UNIT, "cores": leg["cores"], "kind": "oracle", "sample": leg["sample"],
               "ms_per_step_of_sample": leg["ms_per_step"],
               "append_prefill_tokens_per_s": leg["append_prefill_tokens_per_s"]}

    if rank == 0:
        cfg = workload_config(wl, cold, L * resident_mean)
        if args.uniform_bits:
            cfg["uniform_bits"] = args.uniform_bits
        if args.scale_groups != 1:
            cfg["scale_groups"] = args.scale_groups
        line = {
            "metric": METRIC, "value": bytes_job / (ms_step * 1e-3) / 1e9, "unit": UNIT,
            "n_gpus": world, "steps": K_steps, "warmup": W, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": cfg,
            "clocks": clocks,
            "e2e": {"value": bytes_job / (ms_e2e * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms_e2e,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches_timed),
            "roofline": {"bound": "hbm", "kernel": "k_decode_attn", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_kind": "of " + peak_kind,
                         "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH if is_headline and B == 16 and ctx_len == 32768 else None,
                         "algorithmic_bytes_per_launch": dec_bytes,
                         "avg_launch_us": ms_attn * 1e3,
                         "timed_in": ("the timed steps, one event pair per launch" if cold else
                                      "a second pass of the same number of steps with an event pair around every launch"),
                         "frac_with_index_bytes": (dec_bytes + index_bytes) / (ms_attn * 1e-3) / 1e9 / peak},
            "cpu_baseline": cpu,
            "decode_attn_us_per_layer": ms_attn * 1e3,
            "step_us": ms_step * 1e3,
            "step_us_warm_l2": None if ms_warm is None else ms_warm * 1e3,
            "step_us_with_kernel_events": None if ms_instrumented is None else ms_instrumented * 1e3,
            "append_prefill_tokens_per_s": {
                "controller_fused": B * ctx_len / (ms_prefill_fused * 1e-3),
                "bits_given": B * ctx_len / (ms_prefill_given * 1e-3),
                "ms_fused": ms_prefill_fused, "ms_bits_given": ms_prefill_given,
                "GBps_fused": (B * ctx_len * Hkv * 256 + ctl_written) / (ms_prefill_fused * 1e-3) / 1e9,
                "GBps_bits_given": (B * ctx_len * Hkv * 256 + given_written) / (ms_prefill_given * 1e-3) / 1e9,
                "controller_class_histogram": ctl_hist, "note": "one layer"},
            "memory": {"packed_row_bytes": int(L * resident1), "arena_bytes_in_use": int(arena_used * arena_block),
                       "arena_bytes_reserved": int(arena_total * arena_block),
                       "fp16_cache_bytes": int(L * B * Hkv * (ctx_len + step_no[0]) * 256),
                       "note": "arena blocks are taken on demand; kvq_create reserves the worst case, "
                               "kvq_create_arena any budget"},
            "kv_bytes_per_layer": dec_bytes, "expected_bits": ebits,
            "device_bytes": kq.kvq_device_bytes(ctx), "input_generation_s": t_gen,
        }
        print(json.dumps(line))
    kq.kvq_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
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
    ap.add_argument("--batch", type=int, default=0,
                    help="fewer sequences than the workload's 16, likewise for profiler captures only")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    wl = synth.CONFIGS[args.workload]
    if args.context > 0:
        wl = dataclasses.replace(wl, context=args.context, name="%s-context-%d" % (wl.name, args.context))
    if args.batch > 0:
        wl = dataclasses.replace(wl, batch=args.batch, name="%s-batch-%d" % (wl.name, args.batch))
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
