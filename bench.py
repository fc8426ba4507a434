#!/usr/bin/env python
"""Benchmark of the verify-and-resample pass (one step = one pass over one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config C]

Prints ONE JSON line.  Metric: verified draft positions per second (sum of K_b over the
batch, divided by the time of one pass), whole job over all ranks.  `value` is measured
with the inputs resident in HBM; `e2e` is the same metric through the host-buffer entry
point, with host<->device copies inside the timed region.  `roofline` relates the dominant
kernel to the measured HBM copy bandwidth; `cpu_baseline` is the fp64 oracle on the host.
For N > 1 (torchrun) every rank verifies its own full-size batch: the path shards by
sequence and needs no collective, so scaling is weak.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "verified_draft_positions_per_s"
UNIT = "positions/s"
FALLBACK_HBM_GBS = 6650.0
L2_BYTES = 126 * 1024 * 1024

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the dominant
# kernel from the ncu capture summarised under profiles/; only valid for the kernel source
# it was taken from (sha256 of the files that kernel is compiled from), otherwise reported as null.
NCU_TRAFFIC = {"csrc_sha256": "1e214ecf62836d7d13fa6d3a5675307fc503a6c3f67182c204e3c336a43bbe13",
               "workload": "config3 capture of specv_ring_stats (279.14 MB read + 4.14 MB written for 279.09 MB of logits) scaled by logit bytes to config5", "bytes_per_launch": 2424588446}


# kernel set of a pass as spec_verify_last_path reports it
PATH_NAMES = {1: "streaming", 2: "ring", 3: "cluster"}


# the sources the dominant kernel (specv_ring_stats) is compiled from
DOMINANT_KERNEL_SOURCES = ("specv_device.cuh", "specv_stream_kernels.cuh", "specv_ring_kernels.cuh")


def csrc_sha256() -> str:
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2411_00853_b200", "csrc")
    for name in DOMINANT_KERNEL_SOURCES:
        h.update(open(os.path.join(d, name), "rb").read())
    return h.hexdigest()


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML (read-only)."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, torch_device_index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons = [], 0
        self.by_region = {}
        self.region_name = None
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self._active = threading.Event()
        self.handle = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None

    def run(self):
        while not self._stop_evt.is_set():
            if self.handle is not None and self._active.is_set():
                try:
                    mhz = int(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM))
                    try:
                        r = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                    except Exception:
                        r = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                    name = self.region_name
                    if name == "main":
                        self.samples.append(mhz)
                        self.reasons |= r
                    reg = self.by_region.setdefault(name, [[], 0])
                    reg[0].append(mhz)
                    reg[1] |= r
                except Exception:
                    pass
            time.sleep(self.period)

    def region(self, on: bool, name: str = "main"):
        """Samples taken while a region is on are filed under its name; "main" is the timed region of
        the headline figure."""
        if on:
            self.region_name = name
            self._active.set()
        else:
            self._active.clear()

    def region_summary(self, name: str):
        mhz, reasons = self.by_region.get(name, [[], 0])
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(v for k, v in self.REASONS.items() if reasons & k), "samples": len(mhz)}

    def stop(self):
        self._stop_evt.set()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(v for k, v in self.REASONS.items() if self.reasons & k),
                "samples": len(self.samples)}


def workload_config(w, cfg):
    return {"workload": f"config{cfg}: {w.recipe}", "B": int(w.B), "V": int(w.V), "logits_dtype": w.dtype,
            "draft_positions": int(w.n_draft_total), "logit_bytes": int(w.logit_bytes),
            "l2": ("L2 flushed between timed iterations (a 252 MB buffer is read)" if needs_flush(w) else
                   "inputs larger than L2 (every pass streams %.0f MB, %.0f times the L2%s)" % (
                       w.logit_bytes / 1e6, w.logit_bytes / L2_BYTES,
                       "; consecutive passes rotate through 3 distinct copies of the logits" if input_sets(w) > 1 else ""))}


def needs_flush(w) -> bool:
    """A workload that fits in L2 is timed with an L2 flush between passes."""
    return w.logit_bytes <= 2 * L2_BYTES


def input_sets(w) -> int:
    """Distinct copies of the logits that consecutive passes rotate through: three for workloads
    between 2 and 8 times the L2 (so that no pass can find lines of its own input left by an
    earlier pass), one otherwise."""
    return 3 if 2 * L2_BYTES < w.logit_bytes < 8 * L2_BYTES else 1


# --------------------------------------------------------------------------- reference arm
def run_reference(args):
    """The fp64 oracle, as it stands, on the host cores: the baseline arm."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2411_00853_b200 import workloads as W
    cores = os.cpu_count() or 1
    # a bounded sample of the workload: the first `n_seq` sequences of the batch, sized so
    # that warm-up + timed steps finish within a few minutes
    spec_B = {1: 1, 2: 8, 3: 64, 4: 256, 5: 512}[args.config]
    n_seq = min(spec_B, max(cores, 16))
    w = W.make_config(args.config, B=n_seq)
    call = lambda: oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, w.k_per_row,
                                      w.temperature, w.uniforms, threads=cores)
    t0 = time.perf_counter(); call(); one = time.perf_counter() - t0
    budget_s = 150.0
    steps = max(1, min(args.steps, int(budget_s / max(one, 1e-3)) - args.warmup))
    for _ in range(min(args.warmup, 2)):
        call()
    t0 = time.perf_counter()
    for _ in range(steps):
        call()
    dt = (time.perf_counter() - t0) / steps
    value = w.n_draft_total / dt
    sample = f"first {n_seq} of {spec_B} sequences of config{args.config} per step ({w.n_draft_total} draft positions)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 2), "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, args.config) | {"sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- our arm
class DeviceWorkload:
    def __init__(self, w, device):
        import torch
        from paper_2411_00853_b200 import binding
        self.w = w
        as_t = lambda a: torch.from_numpy(a).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        self.host = dict(target=as_t(w.target_logits), draft=as_t(w.draft_logits),
                         tokens=torch.from_numpy(w.draft_tokens), k=torch.from_numpy(np.ascontiguousarray(w.k_per_row)),
                         temperature=torch.from_numpy(np.ascontiguousarray(w.temperature)),
                         uniforms=torch.from_numpy(np.ascontiguousarray(w.uniforms)))
        self.dev = {k: v.to(device) for k, v in self.host.items()}
        # consecutive passes rotate through these copies of the logits (see input_sets)
        self.logit_sets = [(self.dev["target"], self.dev["draft"])]
        for _ in range(input_sets(w) - 1):
            self.logit_sets.append((self.dev["target"].clone(), self.dev["draft"].clone()))
        self.calls = 0
        D, B, V = w.n_draft_total, w.B, w.V
        self.accepted = torch.empty(B, dtype=torch.int32, device=device)
        self.emitted = torch.empty(D + B, dtype=torch.int32, device=device)
        self.workspace = torch.empty(max(256, binding.workspace_bytes(B, D, V)), dtype=torch.uint8, device=device)
        self.binding = binding
        self.stream = torch.cuda.current_stream(device).cuda_stream
        # a batch whose sequences all have the same lookahead is passed the way a caller with a
        # fixed lookahead would pass it: k_per_row = NULL, k_uniform = K
        k = np.asarray(w.k_per_row)
        self.k_uniform = int(k[0]) if k.size and np.all(k == k[0]) else None

    def step(self):
        d = self.dev
        target, draft = self.logit_sets[self.calls % len(self.logit_sets)]
        self.calls += 1
        self.binding.spec_verify(target, draft, d["tokens"], None if self.k_uniform is not None else d["k"],
                                 d["temperature"], d["uniforms"], k_uniform=self.k_uniform,
                                 accepted_len=self.accepted, emitted_tokens=self.emitted,
                                 workspace=self.workspace, stream=self.stream)


class L2Flush:
    """Evicts the previous pass's lines from L2 by READING a buffer of twice the L2 size (a sum
    over it).  Reading leaves clean lines behind; overwriting the buffer instead would leave the
    L2 full of dirty lines whose write-back (126 MB) is then charged to the pass under test."""
    def __init__(self, device):
        import torch
        self.buf = torch.zeros(2 * L2_BYTES // 4, dtype=torch.int32, device=device)
        self.sink = torch.zeros(1, dtype=torch.int64, device=device)

    def zero_(self):           # the name the timing loops call
        import torch
        torch.sum(self.buf.view(1, -1), dim=(1,), out=self.sink)


def time_steps(dw, steps, warmup, flush=None, barrier=None):
    """Mean ms per step over `steps` passes, CUDA events on the launching stream.  Without a
    flush buffer the passes run back to back inside one event pair; with one, the buffer is
    overwritten before every pass and each pass has its own event pair."""
    return time_steps_stats(dw, steps, warmup, flush, barrier)["mean_ms"]


def time_steps_stats(dw, steps, warmup, flush=None, barrier=None, per_step=True):
    """{"mean_ms", "median_ms", "min_ms"}: the mean as time_steps states it; median and minimum from
    per-pass event pairs (for back-to-back runs taken in a second loop of at most 200 passes)."""
    import torch
    for _ in range(warmup):
        if flush is not None:
            flush.zero_()
        dw.step()
    if barrier:
        barrier()
    torch.cuda.synchronize()

    def each(n):
        # all passes are enqueued at once, an event before and after each: the device-side time
        # of every pass, without the host's launch latency in it
        pairs = []
        for _ in range(n):
            if flush is not None:
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); dw.step(); e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in pairs]

    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            dw.step()
        e1.record()
        torch.cuda.synchronize()
        mean = e0.elapsed_time(e1) / steps
        if barrier:
            barrier()
        singles = each(min(steps, 200)) if per_step else [mean]
    else:
        singles = each(steps)
        mean = float(np.mean(singles))
        if barrier:
            barrier()
    return {"mean_ms": mean, "median_ms": float(np.median(singles)), "min_ms": float(np.min(singles))}


def sustained_run(dw, seconds, ms_estimate, sampler):
    """Back-to-back passes for at least `seconds` inside ONE event pair, with the SM clock sampled
    meanwhile: the figure under the power cap, beside the short-run one."""
    import torch
    n = int(max(50, np.ceil(seconds * 1e3 / ms_estimate)))
    for _ in range(20):
        dw.step()
    torch.cuda.synchronize()
    sampler.region(True, "sustained")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        dw.step()
    e1.record()
    torch.cuda.synchronize()
    sampler.region(False)
    total_ms = e0.elapsed_time(e1)
    return n, total_ms


def kernel_times(dw, steps, flush=None):
    """Mean ms of the three kernels of a pass (prologue, row statistics, resolve), from
    events the library records around its own kernels."""
    import torch
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for e in ev:
        e.record()
    torch.cuda.synchronize()
    dw.binding.set_trace_events(ev)
    acc = np.zeros(3)
    try:
        for _ in range(steps):
            if flush is not None:
                flush.zero_()
            dw.step()
            torch.cuda.synchronize()
            acc += [ev[i].elapsed_time(ev[i + 1]) for i in range(3)]
    finally:
        dw.binding.set_trace_events(None)
    return (acc / steps).tolist()


def graph_replay_us(dw, iters=100):
    """One pass captured in a CUDA graph (after an ordinary call has done the library's lazy
    per-device set-up) and replayed back to back: microseconds per replay, L2 not flushed."""
    import torch
    dw.step()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    keep = dw.stream
    g = torch.cuda.CUDAGraph()
    try:
        with torch.cuda.stream(side):
            dw.stream = side.cuda_stream
            with torch.cuda.graph(g, stream=side):
                dw.step()
    finally:
        dw.stream = keep
    torch.cuda.synchronize()
    for _ in range(5):
        g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e3


class GreedyWorkload:
    """The greedy pass (temperature -> 0) on the target rows and draft tokens of a workload."""
    def __init__(self, dw, w, device):
        import torch
        self.dw, self.binding = dw, dw.binding
        self.accepted = torch.empty(w.B, dtype=torch.int32, device=device)
        self.emitted = torch.empty(w.n_draft_total + w.B, dtype=torch.int32, device=device)
        self.workspace = torch.empty(max(256, dw.binding.greedy_workspace_bytes(w.B, w.n_draft_total)),
                                     dtype=torch.uint8, device=device)

    def step(self):
        d = self.dw.dev
        self.binding.spec_verify_greedy(d["target"], d["tokens"], d["k"], accepted_len=self.accepted,
                                        emitted_tokens=self.emitted, workspace=self.workspace, stream=self.dw.stream)


def greedy_leg(dw, w, device, steps, warmup, flush, peak):
    """Times the greedy pass on the same batch (it reads the target rows only) and checks a sample
    of its output against the oracle, exactly."""
    import oracle
    gw = GreedyWorkload(dw, w, device)
    ms = time_steps(gw, steps, warmup, flush=flush)
    k_ms = kernel_times(gw, min(steps, 50), flush=flush)
    rows = w.n_draft_total + w.B
    row_bytes = w.V * (4 if w.dtype == "f32" else 2)
    n_seq = min(w.B, 64)
    sub = w.take(0, n_seq)
    ora = oracle.spec_verify_greedy(sub.target_logits, sub.draft_tokens, sub.k_per_row, threads=os.cpu_count() or 1)
    acc = gw.accepted.cpu().numpy()[:n_seq]
    em = gw.emitted.cpu().numpy()[:sub.n_draft_total + n_seq]
    exact = bool(np.array_equal(acc, ora.accepted_len) and np.array_equal(em, ora.emitted_tokens))
    gbs = rows * row_bytes / (k_ms[1] * 1e-3) / 1e9
    return {"ms_per_step": ms, "value": w.n_draft_total / (ms * 1e-3), "unit": UNIT,
            "bytes_per_pass": int(rows * row_bytes), "argmax_kernel_ms": k_ms[1], "argmax_kernel_gbs": gbs,
            "argmax_kernel_frac": gbs / peak, "whole_pass_frac": rows * row_bytes / (ms * 1e-3) / 1e9 / peak,
            "path": PATH_NAMES[dw.binding.last_path()],
            "parity_sample": {"sequences": n_seq, "exact": exact},
            "note": "temperature -> 0 limit: accept while the draft token is the target argmax; target rows only"}


def tree_leg(device, steps, warmup, peak):
    """Times tree-structured verification on a seeded batch of draft trees (64 sequences, vocabulary
    128256, bf16) and checks a sample of its output against the oracle."""
    import torch
    import oracle
    from paper_2411_00853_b200 import binding
    from paper_2411_00853_b200 import workloads as W
    w = W.make_tree_config(B=64, V=128256)
    D, B = w.n_draft_total, w.B
    dev = lambda a: (torch.from_numpy(a).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(np.ascontiguousarray(a))).to(device)
    t = dict(tl=dev(w.target_logits), dl=dev(w.draft_logits), tok=dev(w.draft_tokens), par=dev(w.node_parent),
             n=dev(w.k_per_row), T=dev(w.temperature), u=dev(w.uniforms))
    acc = torch.empty(B, dtype=torch.int32, device=device)
    em = torch.empty(D + B, dtype=torch.int32, device=device)
    ws = torch.empty(max(256, binding.tree_workspace_bytes(B, D, w.V)), dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream(device).cuda_stream

    class Step:
        def step(self_inner):
            binding.spec_verify_tree(t["tl"], t["dl"], t["tok"], t["par"], t["n"], t["T"], t["u"], accepted_len=acc,
                                     emitted_tokens=em, workspace=ws, stream=stream)
    ms = time_steps(Step(), steps, warmup)
    n_seq = 16
    sub = w.take(0, n_seq)
    ora = oracle.spec_verify_tree(sub.target_logits, sub.draft_logits, sub.draft_tokens, sub.node_parent, sub.k_per_row,
                                  sub.temperature, sub.uniforms, threads=os.cpu_count() or 1)
    a = acc.cpu().numpy()[:n_seq]
    e = em.cpu().numpy()[:sub.n_draft_total + n_seq]
    same = int(sum(a[b] == ora.accepted_len[b] and np.array_equal(
        e[int(sub.off_t[b]):int(sub.off_t[b]) + int(sub.k_per_row[b]) + 1],
        ora.emitted_tokens[int(sub.off_t[b]):int(sub.off_t[b]) + int(sub.k_per_row[b]) + 1]) for b in range(n_seq)))
    return {"ms_per_step": ms, "nodes": int(D), "sequences": int(B), "value": D / (ms * 1e-3), "unit": "tree nodes/s",
            "bytes_first_pass": int(w.logit_bytes), "first_pass_frac_of_peak": w.logit_bytes / (ms * 1e-3) / 1e9 / peak,
            "path": PATH_NAMES[binding.last_path()],
            "parity_sample": {"sequences": n_seq, "identical": same},
            "note": "every rejected sibling costs one more pass over its context's two rows, so the pass reads "
                    "more than bytes_first_pass; the fraction is a lower bound on the achieved bandwidth"}


def lm_head_leg(w, device, steps, warmup):
    """Times spec_verify_from_hidden on the batch shape of the workload (hidden sizes 4096 for the
    target model and 2048 for the draft model, N(0,1) hidden states, weights N(0, 9/H)): the two
    LM-head products on the tensor cores with the row statistics in their epilogue, then the resolve
    kernel -- against the measured bf16 matmul throughput -- and checks four logits rows against the
    fp64 oracle's product."""
    import torch
    import oracle
    from paper_2411_00853_b200 import binding
    H, Hd, V, B, D = 4096, 2048, int(w.V), int(w.B), int(w.n_draft_total)
    g = torch.Generator(device=device)
    g.manual_seed(7)
    rnd = lambda r, c, s: (torch.randn((r, c), generator=g, device=device, dtype=torch.float32) * s).to(torch.bfloat16)
    th, dh = rnd(D + B, H, 1.0), rnd(D, Hd, 1.0)
    tw, dw = rnd(V, H, 3.0 / H ** 0.5), rnd(V, Hd, 3.0 / Hd ** 0.5)
    d = {k: torch.from_numpy(np.ascontiguousarray(getattr(w, k))).to(device) for k in ("draft_tokens", "k_per_row", "temperature", "uniforms")}
    tl = torch.empty((D + B, V), dtype=torch.bfloat16, device=device)
    dl = torch.empty((D, V), dtype=torch.bfloat16, device=device)
    acc = torch.empty(B, dtype=torch.int32, device=device)
    em = torch.empty(D + B, dtype=torch.int32, device=device)
    ws = torch.empty(binding.from_hidden_workspace_bytes(B, D, V), dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream(device).cuda_stream

    class Fused:
        def step(self_inner):
            binding.spec_verify_from_hidden(th, tw, dh, dw, d["draft_tokens"], d["k_per_row"], d["temperature"], d["uniforms"],
                                            target_logits=tl, draft_logits=dl, accepted_len=acc, emitted_tokens=em,
                                            workspace=ws, stream=stream)

    class Unfused:      # the same products by the vendor library, then the verify pass reading their logits
        def step(self_inner):
            torch.matmul(th, tw.t(), out=tl)
            torch.matmul(dh, dw.t(), out=dl)
            binding.spec_verify(tl, dl, d["draft_tokens"], d["k_per_row"], d["temperature"], d["uniforms"],
                                accepted_len=acc, emitted_tokens=em, workspace=ws, stream=stream)

    fused_ms = time_steps(Fused(), steps, warmup)
    status = binding.from_hidden_status(ws, B, D, V)
    rows = [0, 1, D + B - 1, (D + B) // 2]
    got = tl[rows].float().cpu().numpy().astype(np.float64)
    to_bits = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    want_bits = oracle.lm_head(to_bits(th[rows]), to_bits(tw), threads=os.cpu_count() or 1)
    want = (want_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.maximum(np.abs(want), np.abs(got)), 1e-30))) - 7)
    within = bool(np.all(np.abs(got - want) <= ulp * 1.0001 + 1e-4))
    unfused_ms = time_steps(Unfused(), steps, warmup)
    flops = 2.0 * V * ((D + B) * H + D * Hd)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak = float(peaks.get("bf16_tflops_sustained", 1400.0))
    return {"ms_per_step": fused_ms, "tflops": flops / (fused_ms * 1e-3) / 1e12,
            "frac_of_measured_bf16_sustained": flops / (fused_ms * 1e-3) / 1e12 / peak, "peak_tflops": peak,
            "peak_source": "measured (sustained cuBLAS bf16)" if "bf16_tflops_sustained" in peaks else "fallback",
            "shape": {"target_rows": D + B, "draft_rows": D, "V": V, "H_target": H, "H_draft": Hd},
            "vendor_matmuls_then_spec_verify_ms": unfused_ms,
            "status_word": status,
            "parity_sample": {"logit_rows": len(rows), "within_one_bf16_ulp_of_fp64_product": within,
                              "exactly_equal_frac": float((got == want).mean())},
            "note": "logits written once and never read back for the statistics; resolve kernel re-reads <= 2 rows per sequence"}


def run_ours(args):
    import torch
    from paper_2411_00853_b200 import binding, sharding
    from paper_2411_00853_b200 import workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    binding.load()
    binding.set_path({"auto": 0, "streaming": 1, "ring": 2}[args.path])
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    barrier = (lambda: dist.barrier()) if dist else None

    w = W.make_config(args.config)
    dw = DeviceWorkload(w, device)
    flush_buf = L2Flush(device)
    flush = flush_buf if needs_flush(w) else None

    sampler = ClockSampler(local)
    sampler.start()
    sampler.region(True)
    launches0 = binding.launch_count()
    timing = time_steps_stats(dw, args.steps, args.warmup, flush=flush, barrier=barrier, per_step=False)
    launches = binding.launch_count() - launches0
    launches_timed = launches * args.steps // (args.steps + args.warmup)
    ms = sharding.max_over_ranks(timing["mean_ms"], device)
    sampler.region(False)
    per_pass = time_steps_stats(dw, min(args.steps, 200), 0, flush=flush) if flush is None else timing
    sampler.region(True)
    k_steps = min(args.steps, 50)
    k_ms = kernel_times(dw, k_steps, flush=flush)

    # end to end: host buffers through spec_verify_host, copies inside the timed region
    pinned = {k: v.pin_memory() for k, v in dw.host.items()}
    arena = torch.empty(binding.host_arena_bytes({"f32": binding.F32, "bf16": binding.BF16, "f16": binding.F16}[w.dtype], w.B,
                                                 w.n_draft_total, w.V), dtype=torch.uint8, device=device)
    acc_h = torch.empty(w.B, dtype=torch.int32).pin_memory()
    em_h = torch.empty(w.n_draft_total + w.B, dtype=torch.int32).pin_memory()

    def e2e_step():
        binding.spec_verify_host(pinned["target"], pinned["draft"], pinned["tokens"], pinned["k"],
                                 pinned["temperature"], pinned["uniforms"], arena,
                                 accepted_len=acc_h, emitted_tokens=em_h, stream=dw.stream)
    e2e_steps = max(3, min(args.steps, 30))
    for _ in range(3):
        e2e_step()
    if barrier:
        barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    e2e_ms = sharding.max_over_ranks(e2e_ms, device)
    sampler.region(False)
    h2d = sum(v.numel() * v.element_size() for v in pinned.values())
    d2h = acc_h.numel() * 4 + em_h.numel() * 4
    del pinned, arena
    torch.cuda.empty_cache()

    positions = w.n_draft_total * world
    peak, peak_kind = measured_peak_gbs()
    stats_ms = k_ms[1]
    ring = binding.last_path() == 2
    # the ring kernel set has no prologue kernel (its statistics kernel does that work): the
    # first interval is then only the gap between two event records
    names = {1: ["specv_prologue", "specv_row_stats", "specv_resolve"],
             2: ["(event gap)", "specv_ring_stats", "specv_ring_resolve"],
             3: ["(event gap)", "specv_cluster_pass", "(event gap after)"]}[binding.last_path()]
    traffic = (NCU_TRAFFIC["bytes_per_launch"]
               if ring and args.config == 5 and NCU_TRAFFIC["csrc_sha256"] == csrc_sha256() else None)
    achieved = w.logit_bytes / (stats_ms * 1e-3) / 1e9
    # special-function work: one base-2 exponential per logit in the statistics kernel; in the resolve
    # kernel one per element of every row a token is drawn from (two rows at a rejection, one otherwise)
    elt = 4 if w.dtype == "f32" else 2
    acc_now = dw.accepted.cpu().numpy()
    resolve_rows = int(sum(2 if int(a) < int(k) else 1 for a, k in zip(acc_now, w.k_per_row)))
    line = {
        "metric": METRIC, "value": positions / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": workload_config(w, args.config),
        "clocks": sampler.summary(),
        "e2e": {"value": positions / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms, "steps": e2e_steps},
        "gpu_launches": int(launches_timed),
        "roofline": {"bound": "hbm", "kernel": names[1], "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                     "traffic_note": ("extrapolated from the ncu capture summarised under profiles/ (" +
                                      NCU_TRAFFIC["workload"] + ")") if traffic else
                                     "null: the kernel sources differ from those the ncu capture under profiles/ was taken on",
                     "peak_source": peak_kind + " copy bandwidth (read + write); a read-only stream can exceed it",
                     "kernel_ms": stats_ms, "bytes_per_launch": int(w.logit_bytes),
                     "whole_pass_frac": w.logit_bytes / (ms * 1e-3) / 1e9 / peak,
                     "frac_of_8000_datasheet": achieved / 8000.0,
                     "ex2_per_s": {names[1]: w.logit_bytes / elt / (k_ms[1] * 1e-3),
                                   names[2]: resolve_rows * w.V / (k_ms[2] * 1e-3)}},
        "kernel_ms": {names[0]: k_ms[0], names[1]: k_ms[1], names[2]: k_ms[2]},
        "per_pass": {"median_us": per_pass["median_ms"] * 1e3, "min_us": per_pass["min_ms"] * 1e3,
                     "note": "one event pair per pass (the headline mean is one pair around all passes)"},
    }

    solo = rank == 0 and world == 1
    if solo and not args.no_sustained:
        n, total_ms = sustained_run(dw, args.sustained_seconds, ms, sampler)
        sus_ms = total_ms / n
        clk = sampler.region_summary("sustained")
        line["sustained"] = {
            "passes": n, "seconds": total_ms * 1e-3, "ms_per_step": sus_ms, "value": positions / (sus_ms * 1e-3),
            "unit": UNIT, "whole_pass_frac": w.logit_bytes / (sus_ms * 1e-3) / 1e9 / peak,
            "short_run_whole_pass_frac": w.logit_bytes / (ms * 1e-3) / 1e9 / peak, "clocks": clk,
            "us_times_median_mhz": (sus_ms * 1e3 * clk["sm_mhz"]) if clk["sm_mhz"] else None,
            "short_run_us_times_median_mhz": (ms * 1e3 * line["clocks"]["sm_mhz"]) if line["clocks"]["sm_mhz"] else None,
            "note": "back-to-back passes inside one event pair; sw_power_cap is expected on a long run"}
    sampler.stop()

    if solo and not args.no_early_exit and ring:
        binding.set_early_exit(True)
        ee = time_steps_stats(dw, min(args.steps, 100), args.warmup, flush=flush)
        binding.set_early_exit(False)
        acc_ee = dw.accepted.cpu().numpy()
        em_ee = dw.emitted.cpu().numpy()
        dw.step()
        torch.cuda.synchronize()
        same = bool(np.array_equal(acc_ee, dw.accepted.cpu().numpy()) and np.array_equal(em_ee, dw.emitted.cpu().numpy()))
        needed = sum(2 * min(int(a) + 1, int(k)) + (1 if a == k else 0) for a, k in zip(acc_ee, w.k_per_row))
        line["early_exit"] = {"ms_per_step": ee["mean_ms"], "median_us": ee["median_ms"] * 1e3, "min_us": ee["min_ms"] * 1e3,
                              "value": positions / (ee["mean_ms"] * 1e-3), "unit": UNIT,
                              "rows_needed_frac": needed / (2 * w.n_draft_total + w.B),
                              "parity_sample": {"sequences": int(w.B), "identical_to_normal_mode": same},
                              "note": "rows after a sequence's first clear rejection are not read; same tokens"}
    if solo and not args.no_tree:
        line["tree"] = tree_leg(device, min(args.steps, 50), args.warmup, peak)
    if solo and not args.no_greedy:
        line["greedy"] = greedy_leg(dw, w, device, min(args.steps, 100), args.warmup, flush, peak)
    if solo and not args.no_lm_head and w.dtype == "bf16":
        line["lm_head"] = lm_head_leg(w, device, min(args.steps, 10), 3)
    if solo:
        # verify the timed output against the oracle on a sample of sequences, and time the oracle
        import oracle
        cores = os.cpu_count() or 1
        # sample size: about 20 core-seconds of oracle work, estimated from a 16-sequence probe
        probe = w.take(0, min(16, w.B))
        t0 = time.perf_counter()
        oracle.spec_verify(probe.target_logits, probe.draft_logits, probe.draft_tokens, probe.k_per_row,
                           probe.temperature, probe.uniforms, threads=cores)
        per_seq_core_s = (time.perf_counter() - t0) * min(cores, probe.B) / probe.B
        n_seq = int(min(w.B, max(16, 20.0 / max(per_seq_core_s, 1e-6))))
        sub = w.take(0, n_seq)
        t0 = time.perf_counter()
        ora = oracle.spec_verify(sub.target_logits, sub.draft_logits, sub.draft_tokens, sub.k_per_row,
                                 sub.temperature, sub.uniforms, threads=cores)
        dt = time.perf_counter() - t0
        # the same oracle on ONE thread, on a smaller sample (about 3 s)
        n_one = int(min(n_seq, max(1, 3.0 / max(per_seq_core_s, 1e-6))))
        one = w.take(0, n_one)
        t0 = time.perf_counter()
        oracle.spec_verify(one.target_logits, one.draft_logits, one.draft_tokens, one.k_per_row, one.temperature,
                           one.uniforms, threads=1)
        dt_one = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": sub.n_draft_total / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {n_seq} of {w.B} sequences ({sub.n_draft_total} draft positions), "
                                          f"{dt:.2f} s wall on {cores} threads",
                                "single_thread": {"value": one.n_draft_total / dt_one, "unit": UNIT, "cores": 1,
                                                  "sample": f"first {n_one} sequences ({one.n_draft_total} draft "
                                                            f"positions), {dt_one:.2f} s"}}
        acc = dw.accepted.cpu().numpy()[:n_seq]
        em = dw.emitted.cpu().numpy()
        mism = excused = 0
        for b in range(n_seq):
            K = int(w.k_per_row[b])
            sl = slice(int(w.off_t[b]), int(w.off_t[b]) + K + 1)
            if acc[b] != ora.accepted_len[b] or not np.array_equal(em[sl], ora.emitted_tokens[sl]):
                n = int(ora.accepted_len[b])
                am = ora.accept_margin[int(w.off_d[b]):int(w.off_d[b]) + min(n + 1, K)]
                if (am.size and np.nanmin(am) < 1e-5) or ora.cdf_margin[b] < 1e-5:
                    excused += 1
                else:
                    mism += 1
        line["parity_sample"] = {"sequences": n_seq, "mismatches": mism, "excused_margin_below_1e-5": excused,
                                 "mean_accepted_len": float(acc.mean())}

        if not args.no_all_configs:
            allc = {}
            for c in (1, 2, 3, 4, 5):
                if c == args.config:
                    allc[str(c)] = {"us_per_call": ms * 1e3, "median_us": per_pass["median_ms"] * 1e3,
                                    "min_us": per_pass["min_ms"] * 1e3,
                                    "positions_per_s": w.n_draft_total / (ms * 1e-3),
                                    "logit_gbs": w.logit_bytes / (ms * 1e-3) / 1e9,
                                    "frac_of_peak": w.logit_bytes / (ms * 1e-3) / 1e9 / peak,
                                    "l2_flushed": flush is not None, "input_sets": input_sets(w)}
                    continue
                del dw
                torch.cuda.empty_cache()
                wc = W.make_config(c)
                dw = DeviceWorkload(wc, device)
                fl = flush_buf if needs_flush(wc) else None
                t = time_steps_stats(dw, 60, 5, flush=fl)
                km = kernel_times(dw, 20, flush=fl)
                m = t["mean_ms"]
                allc[str(c)] = {"us_per_call": m * 1e3, "median_us": t["median_ms"] * 1e3, "min_us": t["min_ms"] * 1e3,
                                "positions_per_s": wc.n_draft_total / (m * 1e-3),
                                "logit_gbs": wc.logit_bytes / (m * 1e-3) / 1e9,
                                "frac_of_peak": wc.logit_bytes / (m * 1e-3) / 1e9 / peak,
                                "kernel_us": [x * 1e3 for x in km], "l2_flushed": fl is not None,
                                "input_sets": input_sets(wc),
                                "k_per_row": "NULL (uniform lookahead)" if dw.k_uniform is not None else "device array",
                                "graph_replay_us_no_flush": graph_replay_us(dw),
                                "path": PATH_NAMES[binding.last_path()]}
            line["all_configs"] = allc
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--no-all-configs", action="store_true")
    ap.add_argument("--path", choices=["auto", "streaming", "ring"], default="auto")
    ap.add_argument("--no-greedy", action="store_true", help="skip the extra greedy-verification leg")
    ap.add_argument("--no-tree", action="store_true", help="skip the tree-structured verification leg")
    ap.add_argument("--no-early-exit", action="store_true",
                    help="skip the leg that times the optional early-exit mode (the headline is always the full pass)")
    ap.add_argument("--no-lm-head", action="store_true",
                    help="skip the leg that times the verify pass fed with hidden states (LM-head products fused in front)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the seconds-long back-to-back run")
    ap.add_argument("--sustained-seconds", type=float, default=2.2)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
