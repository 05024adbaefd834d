#!/usr/bin/env python
"""Benchmark of the entropy-gated K-step head hot path (gate -> compaction -> head).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--no-sweep] [--impl reference]

One step = one pass of the whole path over one batch of synthetic draft tokens. Prints one JSON
line: gated draft tokens/s (device-resident inputs), the same through the host-buffer C-ABI call
(`e2e`), the roofline of the dominant kernel (the persistent head kernel, tensor-bound) as a burst
figure (L2 flushed before every step) and as a sustained one (steps back to back for >= 2 s), the
gate's HBM figure, the SM clock the head kernel really ran at (stamped on the device), a `sweep`
over the other workload shapes, and the fp64 CPU oracle timed on a bounded sample (`cpu_baseline`).
`--impl reference` times only that oracle.
With N > 1 (torchrun) every rank runs the same batch shape on its own GPU: no data-path collective.
"""
from __future__ import annotations

import argparse
import ctypes
import gc
import json
import os
import statistics
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "gated draft tokens/sec through K-step head"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 512 << 20
NOMINAL_TFLOPS = 2250.0        # dense bf16, data sheet
NOMINAL_HBM_GBS = 8000.0       # data sheet
# dram__bytes_read.sum + dram__bytes_write.sum of one head_kernel launch, from the ncu captures summarised
# under profiles/ (head_kernel_<workload>.txt); a workload without a capture of the current kernel reports null
TRAFFIC_BYTES = {"cfg4": 37.4e9, "cfg2": 2.76e9}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def quantile_tau(H: np.ndarray, q: float) -> float:
    Hs = np.sort(H[~np.isnan(H)])
    k = int(round(q * len(Hs)))
    if k <= 0:
        return -1.0
    if k >= len(Hs):
        return float(Hs[-1]) + 1.0
    return 0.5 * (float(Hs[k - 1]) + float(Hs[k]))


# ----------------------------------------------------------------------------------------------
# CPU oracle legs (the only places that touch oracle/)
# ----------------------------------------------------------------------------------------------
def oracle_step(wl, weights, m):
    """Oracle gate + head on the first m draft tokens; returns (seconds, kept)."""
    import oracle
    feat = synth.features(wl, 0, m)
    cond, noise, t = synth.cond(wl, 0, m), synth.noise(wl, 0, m), synth.t_sched(wl.K)
    H = oracle.entropy(feat)
    tau = quantile_tau(H, wl.filter_q)
    t0 = time.perf_counter()
    _, _, idx, count = oracle.gate(feat, tau)
    oracle.head_sample(weights, cond, noise, t, idx)
    return time.perf_counter() - t0, count


def _omp_set_threads(n: int) -> bool:
    """Thread count of the OpenMP runtime the oracle library is linked against."""
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except OSError:
        return False


def cpu_baseline(wl, weights, m, m_one):
    import oracle
    oracle.build()
    sec, kept = oracle_step(wl, weights, m)
    rec = {"value": m / sec, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
           "sample": f"first {m} draft tokens of {wl.name} ({kept} kept), gate + {wl.K}-step head, "
                     f"fp64, {sec:.2f} s"}
    if m_one > 0 and _omp_set_threads(1):
        sec1, kept1 = oracle_step(wl, weights, m_one)
        _omp_set_threads(oracle.threads())
        rec["one_core"] = {"value": m_one / sec1, "unit": UNIT, "cores": 1,
                           "sample": f"first {m_one} draft tokens of {wl.name} ({kept1} kept), {sec1:.2f} s"}
    return rec


def run_reference(args, wl):
    """--impl reference: the fp64 oracle, as it stands, on this machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    weights = synth.head_weights(wl)
    m = args.ref_tokens
    for _ in range(min(args.warmup, 2)):
        oracle_step(wl, weights, m)
    secs = []
    for _ in range(args.steps):
        s, kept = oracle_step(wl, weights, m)
        secs.append(s)
    per = sum(secs) / len(secs)
    val = m / per
    sample = f"each step: first {m} draft tokens of {wl.name} ({kept} kept), gate + {wl.K}-step head, fp64"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "sample_tokens": m},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU during the timed region (read-only NVML)."""

    def __init__(self, dev_index: int, period_s: float = 0.005):
        import threading
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = None
            try:
                # the NVML handle of the very GPU torch uses (CUDA_VISIBLE_DEVICES may reorder or name UUIDs)
                import torch
                uuid = str(torch.cuda.get_device_properties(dev_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.h = None
            if self.h is None:
                visible = os.environ.get("CUDA_VISIBLE_DEVICES")
                phys = dev_index
                if visible:
                    ids = [v.strip() for v in visible.split(",") if v.strip()]
                    if dev_index < len(ids) and ids[dev_index].isdigit():
                        phys = int(ids[dev_index])
                self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None
            return
        self.period = period_s
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()

    def _run(self):
        nv = self.nv
        names = {"applications_clocks_setting": 0x2, "sw_power_cap": 0x4, "hw_slowdown": 0x8, "sync_boost": 0x10,
                 "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80,
                 "display_clock_setting": 0x100}
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for nm, bit in names.items():
                    if r & bit:
                        self.reasons.add(nm)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_min_mhz": min(self.samples),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


class L2Flush:
    """Between timed iterations: 512 MiB written (every line of L2 replaced), then 256 MiB of other data
    read, so that what L2 holds afterwards is unrelated AND clean. (After the write alone L2 is full of
    dirty lines, and the next kernel pays for their write-back on top of its own traffic.)"""

    def __init__(self, torch, dev):
        self.torch = torch
        self.w = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
        self.r = torch.zeros(L2_FLUSH_BYTES // 2, dtype=torch.uint8, device=dev)

    def fill_(self, v):
        self.w.fill_(v)
        self.torch.max(self.r)


def upload_bf16(torch, bits, dev):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)


class Batch:
    """Device-resident inputs and outputs of one workload shape."""

    def __init__(self, torch, dev, wl):
        self.wl, n = wl, wl.n
        self.feat = torch.empty((n, wl.d), dtype=torch.bfloat16, device=dev)
        slab = 32768
        for r0 in range(0, n, slab):
            self.feat[r0:r0 + slab] = upload_bf16(torch, synth.features(wl, r0, min(slab, n - r0)), dev)
        self.cond = torch.empty((n, wl.Dc), dtype=torch.bfloat16, device=dev)
        self.noise = torch.empty((n, wl.C), dtype=torch.float32, device=dev)
        big = 1 << 17
        for r0 in range(0, n, big):
            m = min(big, n - r0)
            self.cond[r0:r0 + m] = upload_bf16(torch, synth.cond(wl, r0, m), dev)
            self.noise[r0:r0 + m] = torch.from_numpy(synth.noise(wl, r0, m)).to(dev)
        self.mask = torch.empty(n, dtype=torch.uint8, device=dev)
        self.idx = torch.empty(n, dtype=torch.int32, device=dev)
        self.count = torch.zeros(1, dtype=torch.int32, device=dev)
        self.ent = torch.empty(n, dtype=torch.float32, device=dev)
        self.out = torch.zeros((n, wl.C), dtype=torch.float32, device=dev)
        self._H = None

    def entropies(self, ardiff, torch):
        """The gate's own entropies (set-up, untimed): tau for a filter rate is their quantile."""
        if self._H is None:
            ardiff.ardiff_entropy_gate(self.feat, -1.0, self.mask, self.idx, self.count, self.ent)
            torch.cuda.synchronize()
            self._H = self.ent.cpu().numpy().astype(np.float64)
        return self._H


def fractions(pk, tflops=None, gbs=None):
    if tflops is not None:
        return {"tflops": tflops, "frac_measured": tflops / pk["bf16_tflops"], "frac_nominal": tflops / NOMINAL_TFLOPS}
    return {"gbs": gbs, "frac_measured": gbs / pk["hbm_gbs"], "frac_nominal": gbs / NOMINAL_HBM_GBS}


def time_steps(torch, ardiff, b, head, tau, t, flush, stream, reps, warm=2):
    """Median gate / head-kernel / step times of `reps` flushed steps, and the survivor count."""
    gate_ms, head_ms, step_ms, mhz = [], [], [], []
    for i in range(warm + reps):
        flush.fill_(i & 0xff)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record(stream)
        ardiff.ardiff_entropy_gate(b.feat, tau, b.mask, b.idx, b.count, stream=stream)
        e[1].record(stream)
        head.ardiff_head_sample(b.cond, b.noise, t, b.idx, b.count, b.out, stream=stream)
        e[2].record(stream)
        hk = head.last_kernel_ms()
        e[2].synchronize()
        if i >= warm:
            gate_ms.append(e[0].elapsed_time(e[1]))
            step_ms.append(e[0].elapsed_time(e[2]))
            head_ms.append(hk)
            mhz.append(head.last_kernel_clock_mhz(stream))
    if head.status() != 0:
        raise RuntimeError("head kernel reported a device-side timeout")
    med = statistics.median
    return med(gate_ms), med(head_ms), med(step_ms), med(mhz), int(b.count.item())


def sweep_record(pk, wl, K, q, gate_ms, head_ms, step_ms, mhz, S, reps):
    flops = S * wl.flops_per_token(K)
    rec = {"workload": wl.name, "n": wl.n, "K": K, "filtered": q, "survivors": S, "reps": reps,
           "gate_ms": gate_ms, "head_kernel_ms": head_ms, "step_ms": step_ms,
           "tokens_per_s": wl.n / (step_ms * 1e-3),
           "survivor_tokens_per_s": (S / (head_ms * 1e-3)) if head_ms > 0 else None,
           "gate": fractions(pk, gbs=wl.gate_bytes() / (gate_ms * 1e-3) / 1e9),
           "head_sm_mhz": mhz}
    rec["head"] = fractions(pk, tflops=flops / (head_ms * 1e-3) / 1e12) if S > 0 and head_ms > 0 else None
    return rec


def run_sweep(torch, ardiff, dev, pk, flush, stream, main_wl, main_batch, main_head, log):
    """The other workload shapes, a few flushed steps each (medians): cfg2; cfg3 at K = 1, 2, 4, 8; cfg4
    filtered and unfiltered; the 2^20-token gate stress at 0/10/50/90/99 % filtered with the survivors
    running through the cfg2-shaped head."""
    recs = []

    def one(b, head, wl, K, q, reps):
        tau = quantile_tau(b.entropies(ardiff, torch), q)
        g, h, s, mhz, S = time_steps(torch, ardiff, b, head, tau, synth.t_sched(K), flush, stream, reps)
        recs.append(sweep_record(pk, wl, K, q, g, h, s, mhz, S, reps))
        log(f"sweep {wl.name} K={K} filtered={q}: gate {g * 1e3:.1f} us, head {h:.3f} ms, S={S}")

    # cfg4 shares the main line's inputs when it is the main workload
    if main_wl.name == "cfg4":
        one(main_batch, main_head, main_wl, main_wl.K, main_wl.filter_q, 5)
        one(main_batch, main_head, main_wl, main_wl.K, 0.0, 5)
    for name, Ks, qs in (("cfg2", [4], [None]), ("cfg3", [1, 2, 4, 8], [None]), ("cfg4", [4], [None, 0.0]),
                         ("cfg5", [4], [0.0, 0.1, 0.5, 0.9, 0.99])):
        if name == main_wl.name:
            continue
        wl = synth.workload(name)
        b = Batch(torch, dev, wl)
        head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, max(Ks), wl.n, synth.head_weights(wl))
        head.set_timing(True)
        for K in Ks:
            for q in qs:
                one(b, head, wl, K, wl.filter_q if q is None else q, 3 if name == "cfg5" else 5)
        head.close()
        del b, head
        gc.collect()
        torch.cuda.empty_cache()
    return recs


def run_next_stage(torch, ardiff, dev, pk, flush, stream):
    """Timings of the later-stage entry points (block-prefix gate, threshold statistics, accepted prefix)
    beside the plain gate on the same input: median of 15 calls, L2 flushed before each."""
    recs = []

    def timed(fn, reps=15):
        ts = []
        for i in range(reps + 3):
            flush.fill_(i & 0xff)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            e1.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1))
        return statistics.median(ts)

    def rec(call, shape, ms, nbytes):
        recs.append({"call": call, "shape": shape, "us": ms * 1e3, "gbs": nbytes / (ms * 1e-3) / 1e9,
                     "frac_measured_hbm": nbytes / (ms * 1e-3) / 1e9 / pk["hbm_gbs"]})

    wl = synth.workload("cfg2")
    feat = upload_bf16(torch, synth.features(wl), dev)
    n, d = feat.shape
    mask = torch.empty(n, dtype=torch.uint8, device=dev)
    idx = torch.empty(n, dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int32, device=dev)
    ent = torch.empty(n, dtype=torch.float32, device=dev)
    ardiff.ardiff_entropy_gate(feat, -1.0, mask, idx, count, ent)
    torch.cuda.synchronize()
    tau = quantile_tau(ent.cpu().numpy().astype(np.float64), 0.05)
    by = n * (2 * d + 5) + 4
    shape = f"{n} tokens x {d}"
    rec("ardiff_entropy_gate", shape, timed(lambda: ardiff.ardiff_entropy_gate(feat, tau, mask, idx, count)), by)
    rec("ardiff_entropy_gate_blocks gamma=8", shape,
        timed(lambda: ardiff.ardiff_entropy_gate_blocks(feat, 1, 8, tau, want_row_entropy=False)), by + n // 8 * 4)
    rec("ardiff_entropy_gate_stats", shape, timed(lambda: ardiff.ardiff_entropy_gate_stats(feat, tau)), by + 24)
    rec("ardiff_tau_calibrate", f"{n} entropies", timed(lambda: ardiff.ardiff_tau_calibrate(ent)), 4 * n + 24)
    r_ = torch.rand(n, device=dev)
    ratio = torch.rand(n, device=dev) + 0.5
    rec("ardiff_accept_prefix gamma=8", f"{n} tokens", timed(lambda: ardiff.ardiff_accept_prefix(r_, ratio, 8)),
        8 * n + n // 8 * 4)
    # row widths off the register path: long rows (one pass, running maximum) and a width that is no multiple of 8
    for dd, nn in ((16384, 8192), (8200, 16384), (777, 65536)):
        wl3 = synth.workload("cfg4", n=nn, d=dd)
        f3 = upload_bf16(torch, synth.features(wl3), dev)
        m3 = torch.empty(nn, dtype=torch.uint8, device=dev)
        i3 = torch.empty(nn, dtype=torch.int32, device=dev)
        rec("ardiff_entropy_gate", f"{nn} tokens x {dd}",
            timed(lambda: ardiff.ardiff_entropy_gate(f3, 5.0, m3, i3, count)), nn * (2 * dd + 5) + 4)
    # attention-map-shaped input: 16 rows (heads x query rows) of 1024 keys per token
    wl2 = synth.workload("cfg3", n=4096 * 16)
    feat2 = upload_bf16(torch, synth.features(wl2), dev)
    rec("ardiff_entropy_gate_blocks rows_per_token=16 gamma=8", "4096 tokens x 16 rows x 1024",
        timed(lambda: ardiff.ardiff_entropy_gate_blocks(feat2, 16, 8, 6.0, want_row_entropy=False)),
        feat2.numel() * 2 + 4096 * 5)
    return recs


def run_gpu(args, wl):
    import torch
    import paper_2512_08537_b200 as ardiff
    from paper_2512_08537_b200 import shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    ardiff.lib()  # fails loudly when libardiff.so cannot be loaded
    t_start = time.time()

    def log(msg):
        if rank == 0 and args.verbose:
            print(f"[{time.time() - t_start:6.1f}s] {msg}", file=sys.stderr, flush=True)

    def slowest(ms):
        return shard.max_over_ranks(ms, device=dev) if dist is not None else ms

    # ---- inputs: seeded on the host, resident in HBM before the timed region ----
    wl_r = synth.workload(wl.name, seed=wl.seed + 1000 * rank, K=wl.K, filter_q=wl.filter_q) if world > 1 else wl
    weights = synth.head_weights(wl)
    n = wl.n
    b = Batch(torch, dev, wl_r)
    t = synth.t_sched(wl.K)
    head = ardiff.Head(wl.C, wl.Dc, wl.W, wl.L, wl.F, wl.K, n, weights)
    head.set_timing(True)
    if args.no_coop:
        head.set_cooperative(False)
    tau = quantile_tau(b.entropies(ardiff, torch), wl.filter_q)
    flush = L2Flush(torch, dev)
    stream = torch.cuda.current_stream()
    log("inputs resident")

    # ---- the gate by itself (gate + compaction launches), flushed before each call; taken before any head
    # kernel has run, so that the SM clock is the one this kernel gets on its own, not what the head's power
    # draw leaves behind ----
    gate_alone = []
    for i in range(23):
        flush.fill_(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        ardiff.ardiff_entropy_gate(b.feat, tau, b.mask, b.idx, b.count, stream=stream)
        e1.record(stream)
        e1.synchronize()
        if i >= 3:
            gate_alone.append(e0.elapsed_time(e1))
    gate_alone_ms = statistics.median(gate_alone)

    warm = max(args.warmup, 3)
    for _ in range(warm):
        flush.fill_(1)
        ardiff.ardiff_entropy_gate(b.feat, tau, b.mask, b.idx, b.count, stream=stream)
        head.ardiff_head_sample(b.cond, b.noise, t, b.idx, b.count, b.out, stream=stream)
    torch.cuda.synchronize()
    if head.status() != 0:
        raise RuntimeError("head kernel reported a device-side timeout")
    S = int(b.count.item())

    # ---- the timed region: `steps` steps, L2 flushed before each (the flush is not timed) ----
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    head_ms, head_mhz, launches = [], [], 0
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    for i in range(args.steps):
        flush.fill_(i & 0xff)
        ev[i][0].record(stream)
        ardiff.ardiff_entropy_gate(b.feat, tau, b.mask, b.idx, b.count, stream=stream)
        launches += ardiff.last_launch_count()
        ev[i][1].record(stream)
        head.ardiff_head_sample(b.cond, b.noise, t, b.idx, b.count, b.out, stream=stream)
        launches += ardiff.last_launch_count()
        ev[i][2].record(stream)
        head_ms.append(head.last_kernel_ms())     # waits for this step's head kernel
        head_mhz.append(head.last_kernel_clock_mhz(stream))
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop() if sampler else None
    gate_ms = [e[0].elapsed_time(e[1]) for e in ev]
    step_ms = [e[0].elapsed_time(e[2]) for e in ev]
    total_ms = slowest(sum(step_ms))
    if head.status() != 0:
        raise RuntimeError("head kernel reported a device-side timeout")
    ms_per_step = total_ms / args.steps
    value = world * n / (ms_per_step * 1e-3)
    log(f"burst: {ms_per_step:.3f} ms/step")

    # ---- sustained: steps back to back for >= 2 s (inputs are larger than L2; no flush, no host sync) ----
    sus_iters = max(10, int(2200.0 / ms_per_step))
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(sus_iters):
        ardiff.ardiff_entropy_gate(b.feat, tau, b.mask, b.idx, b.count, stream=stream)
        head.ardiff_head_sample(b.cond, b.noise, t, b.idx, b.count, b.out, stream=stream)
    e1.record(stream)
    e1.synchronize()
    sus_ms = slowest(e0.elapsed_time(e1)) / sus_iters
    sus_head_ms = head.last_kernel_ms()           # the last launch of the loop, at the settled clock
    sus_mhz = head.last_kernel_clock_mhz(stream)
    sus_clocks = sampler.stop() if sampler else None
    if head.status() != 0:
        raise RuntimeError("head kernel reported a device-side timeout")
    log(f"sustained: {sus_ms:.3f} ms/step over {sus_iters} steps")

    # ---- e2e: the host-buffer C-ABI calls; host<->device copies inside the timed region ----
    # (1) blocking: one ardiff_pipeline_run_host per step, each step timed by itself.
    # (2) overlapped: ardiff_pipeline_submit / _wait over three slots, timed as one region from the first
    #     submit to the last result on the host; the L2 flush sits on the caller's stream before each
    #     submit (inside the region), and each batch starts after it.
    NS = 3
    pipe = ardiff.Pipeline(head, n, wl.d, slots=NS)
    feat_pin = torch.empty((n, wl.d), dtype=torch.bfloat16).pin_memory()
    feat_pin.copy_(b.feat)
    cond_pin = torch.empty((n, wl.Dc), dtype=torch.bfloat16).pin_memory()
    cond_pin.copy_(b.cond)
    noise_pin = torch.empty((n, wl.C), dtype=torch.float32).pin_memory()
    noise_pin.copy_(b.noise)
    out_pin = [torch.empty((n, wl.C), dtype=torch.float32).pin_memory() for _ in range(NS)]
    mask_pin = [torch.empty(n, dtype=torch.uint8).pin_memory() for _ in range(NS)]
    blk_steps = max(3, min(args.steps, 8))
    for _ in range(2):
        pipe.ardiff_pipeline_run_host(feat_pin, cond_pin, noise_pin, tau, t, out_pin[0], mask_pin[0], stream=stream)
    blk_ms = []
    for _ in range(blk_steps):
        flush.fill_(3)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        kept = pipe.ardiff_pipeline_run_host(feat_pin, cond_pin, noise_pin, tau, t, out_pin[0], mask_pin[0],
                                             stream=stream)
        e1.record(stream)
        e1.synchronize()
        blk_ms.append(e0.elapsed_time(e1))
    blk_total = slowest(sum(blk_ms))

    def overlapped(steps):
        for i in range(steps):
            slot = i % NS
            if i >= NS:
                pipe.ardiff_pipeline_wait(slot)
            flush.fill_(i & 0xff)
            pipe.ardiff_pipeline_submit(slot, feat_pin, cond_pin, noise_pin, tau, t, out_pin[slot], mask_pin[slot],
                                        stream=stream)
        kept_last = [pipe.ardiff_pipeline_wait(s) for s in range(NS)]
        pipe.ardiff_pipeline_join(stream)
        return kept_last

    overlapped(2 * NS)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    e2e_steps = max(4, min(args.steps, 30))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    kept_last = overlapped(e2e_steps)
    e1.record(stream)
    e1.synchronize()
    torch.cuda.synchronize()
    if kept_last != [kept] * NS or kept != S or head.status() != 0:
        raise RuntimeError("host-buffer pipeline result differs from the device-resident run")
    e2e_total = slowest(e0.elapsed_time(e1))
    e2e_value = world * n / (e2e_total / e2e_steps * 1e-3)
    blk_value = world * n / (blk_total / blk_steps * 1e-3)
    h2d = n * (2 * wl.d + 2 * wl.Dc + 4 * wl.C)
    d2h = n * (4 * wl.C + 1) + 4
    pipe.close()
    del feat_pin, cond_pin, noise_pin, out_pin, mask_pin
    log(f"e2e: {e2e_total / e2e_steps:.3f} ms/step overlapped, {blk_total / blk_steps:.3f} blocking")

    if rank == 0:
        pk = peaks()
        hk_ms = statistics.mean(head_ms)
        flops = S * wl.flops_per_token()
        achieved = flops / (hk_ms * 1e-3) / 1e12
        sus_achieved = flops / (sus_head_ms * 1e-3) / 1e12
        g_ms = statistics.mean(gate_ms)
        gate_gbs = wl.gate_bytes() / (g_ms * 1e-3) / 1e9
        if clocks is not None:
            clocks["head_kernel_sm_mhz"] = statistics.median(head_mhz)
            clocks["note"] = ("sm_mhz: NVML samples (5 ms period); head_kernel_sm_mhz: SM cycles / wall time "
                              "stamped inside the head kernel, median over the timed steps")
        traffic = TRAFFIC_BYTES.get(wl.name)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "tokens_per_gpu": n, "survivors": S, "d": wl.d, "C": wl.C,
                       "Dc": wl.Dc, "W": wl.W, "L": wl.L, "K": wl.K, "tau": tau,
                       "l2": "512 MiB written, then 256 MiB of other data read, between timed iterations",
                       "parallelism": f"dp{world}"},
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": achieved / pk["bf16_tflops"], "frac_nominal": achieved / NOMINAL_TFLOPS,
                         "nominal_peak": NOMINAL_TFLOPS,
                         "traffic": traffic,
                         "traffic_note": (None if traffic is not None else
                                          "no ncu capture of the current kernel on this workload"),
                         "kernel": "head_kernel", "peak_source": f"{pk['source']} burst bf16",
                         "kernel_ms": hk_ms, "flops_per_launch": flops,
                         "sustained": {"achieved": sus_achieved, "kernel_ms": sus_head_ms,
                                       "peak": pk.get("bf16_tflops_sustained"),
                                       "frac": (sus_achieved / pk["bf16_tflops_sustained"]
                                                if pk.get("bf16_tflops_sustained") else None),
                                       "frac_of_burst_peak": sus_achieved / pk["bf16_tflops"],
                                       "achieved_from_step": flops / (sus_ms * 1e-3) / 1e12,
                                       "ms_per_step": sus_ms, "steps": sus_iters,
                                       "tokens_per_s": world * n / (sus_ms * 1e-3),
                                       "head_kernel_sm_mhz": sus_mhz, "clocks": sus_clocks,
                                       "note": "steps back to back for >= 2 s, no flush (inputs exceed L2); "
                                               "kernel_ms is the last launch of the loop"}},
            "gate": {"bound": "hbm", "achieved": gate_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": gate_gbs / pk["hbm_gbs"], "frac_nominal": gate_gbs / NOMINAL_HBM_GBS,
                     "nominal_peak": NOMINAL_HBM_GBS, "ms": g_ms,
                     "note": "gate + compaction launches, timed inside the steps (right before the head kernel, at "
                             "the clock the power cap leaves)",
                     "isolated": {"ms": gate_alone_ms,
                                  "achieved": wl.gate_bytes() / (gate_alone_ms * 1e-3) / 1e9,
                                  "frac": wl.gate_bytes() / (gate_alone_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                                  "frac_nominal": wl.gate_bytes() / (gate_alone_ms * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                                  "note": "the same two launches alone, before any head kernel has run (SM clock not yet held "
                                          "down by the power cap), L2 flushed before each, median of 20"}},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_total / e2e_steps, "steps": e2e_steps,
                    "mode": "ardiff_pipeline_submit/_wait, 3 slots: copies overlap the kernels of the "
                            "neighbouring steps; L2 flush on the caller's stream inside the region",
                    "blocking": {"value": blk_value, "ms_per_step": blk_total / blk_steps, "steps": blk_steps,
                                 "mode": "ardiff_pipeline_run_host, one step at a time"}},
            "gpu_launches": launches,
            "clocks": clocks,
        }
        # the extra legs must never cost the main line: a failure is recorded in its place
        if world == 1 and not args.no_sweep:
            try:
                line["sweep"] = run_sweep(torch, ardiff, dev, pk, flush, stream, wl, b, head, log)
            except Exception as e:  # noqa: BLE001
                line["sweep"] = {"error": f"{type(e).__name__}: {e}"}
            try:
                line["next_stage"] = run_next_stage(torch, ardiff, dev, pk, flush, stream)
            except Exception as e:  # noqa: BLE001
                line["next_stage"] = {"error": f"{type(e).__name__}: {e}"}
        if world == 1 and not args.no_cpu_baseline:
            try:
                line["cpu_baseline"] = cpu_baseline(wl, weights, args.cpu_tokens, args.cpu_tokens_one_core)
            except Exception as e:  # noqa: BLE001
                line["cpu_baseline"] = {"error": f"{type(e).__name__}: {e}", "kind": "oracle"}
        print(json.dumps(line), flush=True)
    head.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--K", type=int, default=None, help="override the number of sampler steps")
    ap.add_argument("--filter", type=float, default=None, help="override the fraction of tokens dropped")
    ap.add_argument("--cpu-tokens", type=int, default=1024, help="draft tokens of the cpu_baseline sample")
    ap.add_argument("--cpu-tokens-one-core", type=int, default=64, help="draft tokens of its one-core leg (0: skip)")
    ap.add_argument("--ref-tokens", type=int, default=96, help="draft tokens per --impl reference step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the sweep over the other workload shapes")
    ap.add_argument("--no-coop", action="store_true",
                    help="launch the head kernel without the cooperative attribute (for profilers)")
    ap.add_argument("--verbose", action="store_true")
    args = ap.parse_args()
    over = {}
    if args.K is not None:
        over["K"] = args.K
    if args.filter is not None:
        over["filter_q"] = args.filter
    wl = synth.workload(args.workload, **over)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_gpu(args, wl)


if __name__ == "__main__":
    main()
