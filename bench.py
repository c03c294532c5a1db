"""Benchmark of the exit-head hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c1] [--no-extra]

A step is one pass of the whole hot path over one batch: LayerNorm + head projection + entropy / argmax /
max-prob + exit decision for every head of the workload, compaction of the rows that did not exit, and
the DSSD draft-length / accepted-prefix count.  The headline workload is the Pythia-410M-shaped decode
batch (d = 1024, V = 50304, three heads, M = 64 rows).  `value` counts head evaluations of a row per
second (a row through three heads counts three times), which is what the HBM roofline of one head call
bounds: M / (bytes of W / bandwidth).

Prints one JSON line.  With --impl reference the same metric is measured for the fp64 CPU oracle.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "exit-head tokens/s (LN+head+entropy+exit)"
UNIT = "tokens/s"
FALLBACK_PEAKS = dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"]))), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)), reasons=sorted(reasons), samples=len(sm))


# --------------------------------------------------------------------------------------------- workloads


def _algorithmic(M, d, V):
    """Bytes and flops one head call must move / do: W once, h once, 13 bytes of output per row."""
    return 2.0 * V * d + 2.0 * M * d + 13.0 * M, 2.0 * M * V * d


class Workload:
    """Device tensors of one workload and a `step()` that runs the whole hot path once."""

    def __init__(self, name: str, M: int | None, seed: int, n_copies: int, path: int = 0, multi: bool = True):
        import torch
        import paper_2407_21082_b200 as ee
        self.torch, self.ee = torch, ee
        self.path = path
        self.multi = multi and path == 0
        cfg = gen.make_config(name, seed=seed, planted=False, M=M)
        self.name, self.cfg = name, cfg
        self.M, self.d, self.V = cfg["M"], cfg["d"], cfg["V"]

        def bf16(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

        self.heads = []
        for hd in cfg["heads"]:
            dev = dict(gamma=torch.from_numpy(hd["gamma"]).cuda(), beta=torch.from_numpy(hd["beta"]).cuda(), W=[bf16(hd["W"])])
            for _ in range(n_copies - 1):          # distinct copies of W so that consecutive calls miss in L2
                dev["W"].append(dev["W"][0].clone())
            self.heads.append(dev)
        if name == "c3":
            self.h = [bf16(cfg["h_draft"]), bf16(cfg["h_verify"])]
            self.S, self.k = cfg["S"], cfg["k"]
        else:
            self.h = [bf16(cfg["h"])] * len(self.heads)
            self.k = 8
            self.S = self.M // self.k
        self.tau = torch.from_numpy(cfg["tau_per_row"]).cuda() if "tau_per_row" in cfg else float(cfg["tau"])
        # one prepared plan for all heads of the step (a single head included): a call only launches
        ws_bytes = max(ee.ee_exit_head_workspace_bytes(self.M, self.d, self.V),
                       ee.ee_exit_head_multi_workspace_bytes(len(self.heads), self.M, self.d, self.V))
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        ee.ee_workspace_init(self.ws)
        self.outs = [ee.new_outputs(self.M) for _ in self.heads]
        self.comp = dict(kept_idx=torch.empty(self.M, dtype=torch.int32, device="cuda"),
                         kept_count=torch.zeros(1, dtype=torch.int32, device="cuda"),
                         h_out=torch.empty((self.M, self.d), dtype=torch.bfloat16, device="cuda"))
        self.acc = {n: torch.empty(max(self.S, 1), dtype=torch.int32, device="cuda") for n in ("draft_len", "accept_len", "next_tok")}
        self.calls = 0
        self.n_copies = n_copies
        self.head_launches = ee.ee_exit_head_launches(self.M, self.d, self.V, path)
        heads_launches = (ee.ee_exit_head_multi_launches(len(self.heads), self.M, self.d, self.V) if self.multi
                          else len(self.heads) * self.head_launches)
        self.launches_per_step = heads_launches + 1          # + one launch for compaction and accept together
        self.bytes_per_call, self.flops_per_call = _algorithmic(self.M, self.d, self.V)
        self.w_bytes_total = sum(w.numel() * 2 for hd in self.heads for w in hd["W"])
        self.prepare()

    def prepare(self):
        """Marshals every call of a step once (the binding's PreparedCall), so the loop is a few C calls."""
        ee = self.ee
        if self.multi:       # all heads of the step in one call
            self.head_calls = [[ee.PreparedMulti([dict(h=self.h[i], gamma=hd["gamma"], beta=hd["beta"], W=hd["W"][c],
                                                       tau=self.tau, out=self.outs[i]) for i, hd in enumerate(self.heads)],
                                                 1e-5, self.ws)] for c in range(self.n_copies)]
        else:
            self.head_calls = [[ee.prepare_exit_head(self.h[i], hd["gamma"], hd["beta"], 1e-5, hd["W"][c], self.tau,
                                                     out=self.outs[i], workspace=self.ws, path=self.path)
                                for i, hd in enumerate(self.heads)] for c in range(self.n_copies)]
        self.tail_call = self.prepare_tail(self.h[0])

    def prepare_tail(self, h):
        """Compaction of head 0's survivors (with the gather from `h`) and the DSSD count, in one launch."""
        ee = self.ee
        if self.S == 0:
            return ee.prepare_compact(self.outs[0]["exit_mask"], h, out=self.comp)
        n = self.S * self.k
        return ee.prepare_compact_accept(self.outs[0]["exit_mask"], h, self.outs[0]["argmax"][:n].view(self.S, self.k),
                                         self.outs[0]["exit_mask"][:n].view(self.S, self.k),
                                         self.outs[-1]["argmax"][:n].view(self.S, self.k),
                                         out=dict(compact=self.comp, accept=self.acc))

    def run_heads(self):
        for call in self.head_calls[self.calls % self.n_copies]:
            call()
        self.calls += 1

    def run_tail(self):
        self.tail_call()

    def step(self):
        self.run_heads()
        self.run_tail()

    def check(self):
        """Synchronises and raises if a bounded device-side wait gave up (results would be meaningless)."""
        code = self.ee.ee_query_async_error(self.ws)
        if code != 0:
            raise RuntimeError(f"device-side wait timed out in workload {self.name} (ee_status {code})")


def measure(wl: Workload, steps: int, warmup: int, dist=None, sampler: ClockSampler | None = None,
            min_seconds: float = 2.0) -> dict:
    """Times `steps` whole steps, then the head evaluations of `steps` steps alone, with CUDA events on the
    launching stream -- and repeats both regions, `steps` steps each, until about `min_seconds` of device time
    have been spent on each, so that a short region (a few steps run at boost clock before the power cap bites,
    too short for a clock sample) does not stand alone: the reported time is the median over the repeats, the
    first repeat is reported beside it, and the clocks are sampled across all of them.

    The kernels of a step are chained by programmatic dependent launch, and an event recorded between two
    launches breaks that chain (measured: about 5 us per event), so no region has events inside it: the
    first kind gives the step time (the metric), the second the duration of the dominant launch for the
    roofline.  A last, shorter region with an event pair around the head evaluation of every step is reported
    beside them (`head_call_us_inner_events`) to show what the events cost.
    """
    torch = wl.torch
    for _ in range(warmup):
        wl.step()
    wl.check()

    def region(fn):
        """One timed region: barrier and synchronise on both sides, `steps` calls of fn between two events."""
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(steps):
            fn()
        t1.record()
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        return t0.elapsed_time(t1)

    if sampler:
        sampler.start()
    step_ms = [region(wl.step)]
    repeats = int(min(2000, max(1, np.ceil(min_seconds * 1e3 / max(step_ms[0], 1e-3)))))
    if dist is not None:                                  # every rank must run the same number of regions
        r = torch.tensor([repeats], device="cuda")
        dist.all_reduce(r, op=dist.ReduceOp.MAX)
        repeats = int(r.item())
    for _ in range(repeats - 1):
        step_ms.append(region(wl.step))
    heads_ms = [region(wl.run_heads) for _ in range(repeats)]
    clocks = sampler.stop() if sampler else None
    n_inner = min(steps, 500)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_inner)]
    for a, b in ev:
        a.record()
        wl.run_heads()
        b.record()
        wl.run_tail()
    torch.cuda.synchronize()
    wl.check()
    from paper_2407_21082_b200 import replicas
    n_heads = len(wl.heads)
    # per repeat the time of the slowest rank, then the median over the repeats
    per_repeat = torch.tensor(step_ms, dtype=torch.float64, device="cuda")
    if dist is not None:
        dist.all_reduce(per_repeat, op=dist.ReduceOp.MAX)
    total_ms = float(per_repeat.median().item())
    first_ms = float(per_repeat[0].item())
    agg = replicas.aggregate_timing(total_ms, float(steps * n_heads * wl.M), dist, device="cuda")   # the time is already the slowest rank's
    head_ms = float(np.median(heads_ms))
    inner_ms = sum(a.elapsed_time(b) for a, b in ev)
    return dict(total_ms=total_ms, ms_per_step=total_ms / steps, units_per_s=agg["units_per_s"], repeats=repeats,
                ms_per_step_first_repeat=first_ms / steps, ms_per_step_min=float(per_repeat.min().item()) / steps,
                ms_per_step_max=float(per_repeat.max().item()) / steps,
                head_call_us=1e3 * head_ms / (steps * n_heads),
                head_call_us_first_repeat=1e3 * heads_ms[0] / (steps * n_heads),
                head_call_us_inner_events=1e3 * inner_ms / (n_inner * n_heads),
                # step time minus head time; for millisecond-long steps the head-only regions can run slower than the
                # whole steps (power cap), which would make the difference negative: reported as 0 then
                tail_us=max(0.0, 1e3 * (float(np.median(step_ms)) - head_ms) / steps), clocks=clocks)


# DRAM bytes (read + write) one launch of the dominant kernel moved in the ncu captures summarised under
# profiles/, by (workload, rows).  A figure holds only for the kernel sources it was taken on: it is reported
# while the SHA-256 of those sources still matches and as null afterwards.
CSRC = os.path.join(ROOT, "paper_2407_21082_b200", "csrc")
TRAFFIC = {
    ("c0", 8): dict(bytes=51660544 + 1024, heads_per_launch=1, kernel="exit_head_gemm_kernel<0,0,0>",
                    sources=("gemm_kernel.cu", "gemm_roles.cuh", "common.cuh", "sm100_ptx.cuh", "tensor_map.h"),
                    sha256="a488291a0cc4aeecb15686d269133582178c176f7359e972bd4ce770df7bc3f6", profile="profiles/exit_head_gemm_kernel_c0_c2_c3.md"),
    ("c3", 256): dict(bytes=521739904 + 4609536, heads_per_launch=2, kernel="exit_head_gemm_kernel<0,0,1> (CTA pairs)",
                      sources=("gemm_kernel.cu", "gemm_roles.cuh", "common.cuh", "sm100_ptx.cuh", "tensor_map.h"),
                      sha256="a488291a0cc4aeecb15686d269133582178c176f7359e972bd4ce770df7bc3f6", profile="profiles/exit_head_gemm_kernel_c0_c2_c3.md"),
    ("c1", 64): dict(bytes=309859584 + 3799424, heads_per_launch=3, kernel="exit_head_gemm_kernel<0,0,0>",
                     sources=("gemm_kernel.cu", "gemm_roles.cuh", "common.cuh", "sm100_ptx.cuh", "tensor_map.h"),
                     sha256="a488291a0cc4aeecb15686d269133582178c176f7359e972bd4ce770df7bc3f6", profile="profiles/exit_head_gemm_kernel_c1_M64.md"),
    ("c2", 256): dict(bytes=207429248 + 3663872, heads_per_launch=1, kernel="exit_head_gemm_kernel<0,0,1> (CTA pairs)",
                      sources=("gemm_kernel.cu", "gemm_roles.cuh", "common.cuh", "sm100_ptx.cuh", "tensor_map.h"),
                      sha256="a488291a0cc4aeecb15686d269133582178c176f7359e972bd4ce770df7bc3f6", profile="profiles/exit_head_gemm_kernel_c0_c2_c3.md"),
    ("c4", 16384): dict(bytes=1115105024 + 53070080, heads_per_launch=1, kernel="exit_head_gemm_kernel<256,0,1> (CTA pairs)",
                        sources=("gemm_kernel.cu", "gemm_roles.cuh", "common.cuh", "sm100_ptx.cuh", "tensor_map.h"),
                        sha256="a488291a0cc4aeecb15686d269133582178c176f7359e972bd4ce770df7bc3f6", profile="profiles/exit_head_gemm_kernel_c4.md"),
}


def sources_sha256(names) -> str:
    import hashlib
    hsh = hashlib.sha256()
    for n in names:
        with open(os.path.join(CSRC, n), "rb") as f:
            hsh.update(f.read())
    return hsh.hexdigest()


def measured_traffic(wl: "Workload"):
    """(bytes per launch, note) from the committed ncu capture of this workload's dominant kernel, or (None, why)."""
    t = TRAFFIC.get((wl.name, wl.M))
    if t is None or not wl.path == 0:
        return None, "no ncu capture of this workload"
    heads_per_launch = len(wl.heads) if wl.multi else 1
    if heads_per_launch != t["heads_per_launch"]:
        return None, "no ncu capture of this launch shape"
    if sources_sha256(t["sources"]) != t["sha256"]:
        return None, "kernel sources changed since the ncu capture in " + t["profile"]
    return t["bytes"], f"dram read+write of one {t['kernel']} launch ({t['heads_per_launch']} head(s)), {t['profile']}"


def roofline(wl: Workload, head_call_us: float, peaks: dict, src: str) -> dict:
    gbs = wl.bytes_per_call / (head_call_us * 1e-6) / 1e9
    tfs = wl.flops_per_call / (head_call_us * 1e-6) / 1e12
    t_hbm = wl.bytes_per_call / (peaks["hbm_gbs"] * 1e9)
    t_tc = wl.flops_per_call / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_tc:
        return dict(bound="hbm", achieved=round(gbs, 1), peak=peaks["hbm_gbs"], unit="GB/s", frac=round(gbs / peaks["hbm_gbs"], 4),
                    traffic=None, peak_source=f"of {src}", tensor_frac=round(tfs / peaks["bf16_tflops"], 4))
    return dict(bound="tensor", achieved=round(tfs, 1), peak=peaks["bf16_tflops"], unit="TFLOP/s",
                frac=round(tfs / peaks["bf16_tflops"], 4), traffic=None, peak_source=f"of {src} (burst)",
                frac_of_sustained=round(tfs / peaks["bf16_tflops_sustained"], 4), hbm_frac=round(gbs / peaks["hbm_gbs"], 4))


def measure_read_stream(peaks: dict, src: str, gib: float = 1.0, calls: int = 20) -> dict:
    """Rate of a read-only stream over a buffer larger than L2 with the kernels' own weight-streaming mechanism
    (ee_selftest_read_stream), to set beside the copy figure the fractions are quoted against."""
    import torch
    import paper_2407_21082_b200 as ee
    nbytes = int(gib * (1 << 30))
    buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    buf.fill_(1)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    for _ in range(3):
        ee.ee_selftest_read_stream(buf, ws)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(calls):
        ee.ee_selftest_read_stream(buf, ws)
    t1.record()
    torch.cuda.synchronize()
    us = 1e3 * t0.elapsed_time(t1) / calls
    status = ee.ee_query_async_error(ws)
    gbs = nbytes / (us * 1e-6) / 1e9
    return dict(bytes=nbytes, us_per_pass=round(us, 2), gbs=round(gbs, 1), of_copy_peak=round(gbs / peaks["hbm_gbs"], 4),
                peak_source=f"of {src}", status=status,
                note="read-only, one CTA per SM, 12 x 16 KB bulk copies in flight per SM, back-to-back passes over a buffer larger than L2")


# --------------------------------------------------------------------------------------------- e2e and CPU baseline


class E2ESlot:
    """Everything one in-flight step of the host-buffer loop owns: a stream, pinned input rows, staging and result
    buffers, a workspace, and the marshalled calls (one per copy of the weights)."""

    def __init__(self, wl: Workload, stream):
        torch, ee = wl.torch, wl.ee
        S, k = wl.S, wl.k
        self.torch = torch
        self.stream = stream
        self.done = torch.cuda.Event()
        with torch.cuda.stream(stream):       # the binding binds a prepared call to the stream current at its creation
            self.h_host = torch.stack([h.cpu() for h in wl.h]).pin_memory()             # [n_heads, M, d]
            self.ws = torch.empty_like(wl.ws)
            ee.ee_workspace_init(self.ws)
            self.calls = [ee.PreparedMultiHost([dict(gamma=hd["gamma"], beta=hd["beta"], W=hd["W"][c], tau=wl.tau) for hd in wl.heads],
                                               1e-5, self.h_host, self.ws) for c in range(wl.n_copies)]
            self.small_dev = torch.zeros(1 + 3 * max(S, 1), dtype=torch.int32, device="cuda")   # kept_count | draft_len | accept_len | next_tok
            self.small_host = torch.zeros_like(self.small_dev, device="cpu").pin_memory()
            comp = dict(kept_idx=torch.empty_like(wl.comp["kept_idx"]), kept_count=self.small_dev[0:1],
                        h_out=torch.empty_like(wl.comp["h_out"]))
            acc = {n: self.small_dev[1 + i * max(S, 1):1 + (i + 1) * max(S, 1)]
                   for i, n in enumerate(("draft_len", "accept_len", "next_tok"))}
            self.tails = []
            for call in self.calls:
                o = call.out_dev
                if S == 0:
                    self.tails.append(ee.prepare_compact(o[0]["exit_mask"], call.h_dev[0], out=comp))
                else:
                    n = S * k
                    self.tails.append(ee.prepare_compact_accept(o[0]["exit_mask"], call.h_dev[0], o[0]["argmax"][:n].view(S, k),
                                                                o[0]["exit_mask"][:n].view(S, k), o[-1]["argmax"][:n].view(S, k),
                                                                out=dict(compact=comp, accept=acc)))
        stream.synchronize()

    def enqueue(self, c: int):
        """One step: inputs host -> device, the heads, results device -> host, compaction + accept, their counts
        device -> host; all asynchronous on this slot's stream."""
        with self.torch.cuda.stream(self.stream):
            self.calls[c]()
            self.tails[c]()
            self.small_host.copy_(self.small_dev, non_blocking=True)
            self.done.record()

    def read(self) -> int:
        """The caller's read of a finished step: waits for it and touches the results on the host."""
        self.done.synchronize()
        return int(self.small_host[0])

    def error(self, ee) -> int:
        return ee.ee_query_async_error(self.ws)


def run_e2e_loop(wl: Workload, slots, steps: int, warmup: int):
    """steps + warmup steps round-robin over the slots.  With one slot every step is read before the next is
    issued; with two, step i is issued, then step i - 1 is read, so that the host's share of a step (issuing,
    waiting, reading) and its copies overlap the other batch's kernels."""
    torch = wl.torch
    n = len(slots)
    checksum = 0

    def run(count):
        nonlocal checksum
        for it in range(count):
            c = wl.calls % wl.n_copies
            wl.calls += 1
            slots[it % n].enqueue(c)
            if n == 1:
                checksum += slots[0].read()
            elif it >= 1:
                checksum += slots[(it - 1) % n].read()
        if n > 1 and count >= 1:
            checksum += slots[(count - 1) % n].read()

    run(warmup)
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    run(steps)
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    for sl in slots:
        code = sl.error(wl.ee)
        if code != 0:
            raise RuntimeError(f"device-side wait timed out in the end-to-end loop of workload {wl.name} (ee_status {code})")
    return wall, checksum


def measure_e2e(wl: Workload, steps: int, warmup: int) -> dict:
    """The same step through the host-buffer API: every step copies the heads' input rows from pinned host
    memory (one copy), evaluates the heads (ee_exit_head_multi_host), copies the packed results back (one
    copy), runs compaction + accept on the device results, copies their counts back, and the host waits for
    the step and reads its results.  Wall-clock around the loop.  `value` is measured with two independent
    batches in flight (each with its own stream, pinned buffers and workspace; a step's results are read before
    its buffers are used again), `one_batch` with a single batch, where every step is read before the next starts."""
    torch = wl.torch
    n_heads = len(wl.heads)
    slots = [E2ESlot(wl, torch.cuda.Stream()) for _ in range(2)]
    wall1, _ = run_e2e_loop(wl, slots[:1], steps, warmup)
    wall2, _ = run_e2e_loop(wl, slots, steps, warmup)
    call = slots[0].calls[0]
    return dict(value=n_heads * wl.M * steps / wall2, unit=UNIT, h2d_bytes_per_step=call.h2d_bytes,
                d2h_bytes_per_step=call.d2h_bytes + slots[0].small_host.numel() * 4,
                ms_per_step=1e3 * wall2 / steps, batches_in_flight=2,
                one_batch=dict(value=n_heads * wl.M * steps / wall1, ms_per_step=1e3 * wall1 / steps),
                api="ee_exit_head_multi_host + ee_compact_accept per step (three copies), the host waits for each step "
                    "and reads its counts; two independent batches alternate on two streams (their kernels may overlap on the GPU, "
                    "which also fills one batch's dependent-launch bubbles with the other's work)")


def measure_calibration(peaks: dict, src: str, n: int = 1 << 22, calls: int = 30) -> dict:
    """ee_calibrate (threshold of one head from n calibration tokens) timed with CUDA events, and the oracle on
    the same set.  The sort has no fixed algorithmic byte count; `bytes_by_design` is what this implementation's
    passes must move (pack 12 + 8 B, four passes of 8 + 8 + 8 B, two reads of 8 B per token)."""
    import torch
    import oracle
    import paper_2407_21082_b200 as ee
    cs = gen.make_calibration_set(0, n)
    dev = {k: torch.from_numpy(v).cuda() for k, v in cs.items()}
    call = ee.prepare_calibrate(dev["entropy"], dev["argmax_head"], dev["argmax_final"], 0.9)
    for _ in range(3):
        call()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(calls):
        call()
    t1.record()
    torch.cuda.synchronize()
    us = 1e3 * t0.elapsed_time(t1) / calls
    c0 = time.perf_counter()
    ref = oracle.calibrate_threshold(cs["entropy"], oracle.correctness(cs["argmax_head"], cs["argmax_final"]), 0.9)
    cpu_s = time.perf_counter() - c0
    got = call.out if hasattr(call, "out") else None
    counts = got["counts"].cpu().tolist()
    assert counts == [ref["n_exit"], ref["n_correct"], ref["j_hat"]], (counts, ref)
    by_design = (12 + 8 + 4 * 24 + 16) * n
    gbs = by_design / (us * 1e-6) / 1e9
    return dict(n_tokens=n, epsilon=0.9, us_per_call=round(us, 1), tokens_per_s=n / (us * 1e-6), launches=16,
                roofline=dict(bound="hbm", bytes_by_design=by_design, achieved=round(gbs, 1), peak=peaks["hbm_gbs"], unit="GB/s",
                              frac=round(gbs / peaks["hbm_gbs"], 4), peak_source=f"of {src}", traffic=None),
                result=dict(tau=float(got["tau"].item()), n_exit=counts[0], n_correct=counts[1]),
                cpu_baseline=dict(value=n / cpu_s, unit="calibration tokens/s", seconds=round(cpu_s, 3), kind="oracle",
                                  cores=oracle_threads(), sample="the same n tokens (numpy fp64, stable argsort + cumsum)"))


def measure_cascade(peaks: dict, src: str, M: int = 64, calls: int = 300) -> dict:
    """ee_cascade on the c1 shape (three heads in depth order, the last one with tau = +inf playing the full
    model) with planted inputs so that rows do exit; two copies of every W in rotation (cold L2)."""
    import torch
    import oracle
    import paper_2407_21082_b200 as ee
    cfg = gen.make_config("c1", seed=0, planted=True, M=M)
    taus = [1.0, 1.0, float("inf")]

    def bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    h = bf16(cfg["h"])
    ws = torch.empty(ee.ee_cascade_workspace_bytes(M, cfg["d"], cfg["V"]), dtype=torch.uint8, device="cuda")
    ee.ee_workspace_init(ws)
    prepared = []
    for c in range(2):
        heads = [dict(h=h, gamma=torch.from_numpy(hd["gamma"]).cuda(), beta=torch.from_numpy(hd["beta"]).cuda(),
                      W=bf16(hd["W"]), tau=taus[k]) for k, hd in enumerate(cfg["heads"])]
        prepared.append(ee.PreparedCascade(heads, 1e-5, workspace=ws))
    for i in range(6):
        prepared[i % 2]()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for i in range(calls):
        prepared[i % 2]()
    t1.record()
    torch.cuda.synchronize()
    us = 1e3 * t0.elapsed_time(t1) / calls
    out = {k: v.cpu().numpy() for k, v in prepared[(calls - 1) % 2].out.items()}
    c0 = time.perf_counter()
    ref = oracle.cascade([cfg["h"]] * 3, cfg["heads"], taus)
    cpu_s = time.perf_counter() - c0
    same = int((out["exit_head"] == ref["exit_head"]).sum())
    w_bytes = 3 * 2.0 * cfg["V"] * cfg["d"]
    gbs = w_bytes / (us * 1e-6) / 1e9
    return dict(M=M, heads=3, taus=[1.0, 1.0, "inf"], us_per_call=round(us, 2), launches=3 if M <= 512 else 3 * 3, rows_in=out["rows_in"].tolist(),
                rows_per_s=M / (us * 1e-6), rows_agreeing_with_oracle=same,
                roofline=dict(bound="hbm", algorithmic_bytes=w_bytes, achieved=round(gbs, 1), peak=peaks["hbm_gbs"], unit="GB/s",
                              frac=round(gbs / peaks["hbm_gbs"], 4), peak_source=f"of {src}", traffic=None),
                cpu_baseline=dict(value=M / cpu_s, unit="rows/s", seconds=round(cpu_s, 2), kind="oracle", cores=oracle_threads(),
                                  sample=f"the same {M} rows through the same three heads"))


def measure_dssd_round(peaks: dict, src: str, S: int = 32, k: int = 8, rounds: int = 40) -> dict:
    """Whole DSSD rounds (k drafting steps, one verification pass, commit) on the c1 shape, with the hidden states
    coming from a table lookup by the previous token (gen.make_markov_model: the stand-in for the transformer,
    supplied through the driver's callback and run with torch.index_select).  Timed with CUDA events over
    `rounds` rounds; the first round is also run by the oracle."""
    import torch
    import oracle
    import paper_2407_21082_b200 as ee
    spec = gen.CONFIGS["c1"]
    d, V = spec["d"], spec["V"]
    cfg = gen.make_config("c1", seed=0, planted=True, M=4, heads=2)
    planting = gen.make_planting(0, f"c1/planted/d{d}/V{V}", d, V)
    mm = gen.make_markov_model(0, V, d, planting, sigma=0.4)

    def bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    E = [bf16(mm["E_draft"]), bf16(mm["E_verify"])]
    heads = [dict(gamma=torch.from_numpy(hd["gamma"]).cuda(), beta=torch.from_numpy(hd["beta"]).cuda(), W=bf16(hd["W"]))
             for hd in cfg["heads"]]
    heads[0]["tau"] = 1.0
    cap = rounds * (k + 1) + 1
    start = ((np.arange(S, dtype=np.int32) * 1543) % V).astype(np.int32)
    state = dict(last_tok=torch.from_numpy(start).cuda(), out_tok=torch.full((S, cap), -9, dtype=torch.int32, device="cuda"),
                 seq_len=torch.zeros(S, dtype=torch.int32, device="cuda"), finished=torch.zeros(S, dtype=torch.uint8, device="cuda"),
                 stats=torch.zeros(4, dtype=torch.int64, device="cuda"))

    def hidden(tokens, which, h_out):
        torch.index_select(E[which], 0, tokens.long(), out=h_out)

    # the same rounds first with the model as a Python callback (timed on a state of its own), then with the
    # library's table model, which the reported figure and the comparison with the oracle use
    state_py = {n: v.clone() for n, v in state.items()}
    rnd_py = ee.DssdRound(heads[0], heads[1], 1e-5, k, -1, hidden, state_py)
    rnd_py()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(rounds - 1):
        rnd_py()
    t1.record()
    torch.cuda.synchronize()
    us_python_callback = 1e3 * t0.elapsed_time(t1) / (rounds - 1)
    rnd = ee.DssdRound(heads[0], heads[1], 1e-5, k, -1, ee.TableModel(E[0], E[1]), state)
    first = {n: v.clone() for n, v in rnd().items()}
    torch.cuda.synchronize()
    first_len = state["seq_len"].cpu().numpy().copy()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(rounds - 1):
        rnd()
    t1.record()
    torch.cuda.synchronize()
    us = 1e3 * t0.elapsed_time(t1) / (rounds - 1)
    stats = state["stats"].cpu().numpy().tolist()
    ref_state = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    c0 = time.perf_counter()
    ref = oracle.dssd_round(mm["E_draft"], mm["E_verify"], cfg["heads"][0], cfg["heads"][1], 1.0, -1, k, start.copy(), *ref_state)
    cpu_s = time.perf_counter() - c0
    clean = np.ones(S, bool)
    for o in ref["steps"]:
        kp = oracle.decisive_rows(o, 1e-3, 1e-3)
        clean &= kp["argmax"] & kp["exit_mask"]
    clean &= oracle.decisive_rows(ref["verify_out"], 1e-3, 1e-3)["argmax"].reshape(S, k + 1).all(axis=1)
    agree = int((first["accept_len"].cpu().numpy()[clean] == ref["accept_len"][clean]).sum()
                == clean.sum() and (first_len[clean] == ref_state[1][clean]).all())
    w_bytes = (k + 1) * 2.0 * V * d                                       # the heads' weights, once per evaluation
    gbs = w_bytes / (us * 1e-6) / 1e9
    return dict(S=S, k=k, d=d, V=V, tau=1.0, rounds=rounds, us_per_round=round(us, 1), head_evaluations_per_round=k + 1,
                tokens_committed_per_round_per_sequence=round(stats[2] / (rounds * S), 3),
                acceptance_rate=round(stats[1] / max(stats[0], 1), 4), wasted_tokens=stats[0] - stats[1],
                committed_tokens_per_s=stats[2] / rounds / (us * 1e-6),
                first_round_matches_oracle_on_decisive_sequences=bool(agree), decisive_sequences=int(clean.sum()),
                roofline=dict(bound="hbm", algorithmic_bytes=w_bytes, achieved=round(gbs, 1), peak=peaks["hbm_gbs"], unit="GB/s",
                              frac=round(gbs / peaks["hbm_gbs"], 4), peak_source=f"of {src}", traffic=None,
                              note="the stand-in model is the library's table lookup (one small kernel per head evaluation)"),
                us_per_round_python_callback=round(us_python_callback, 1),
                cpu_baseline=dict(value=float(ref_state[3][2]) / cpu_s, unit="committed tokens/s", seconds=round(cpu_s, 2),
                                  kind="oracle", cores=oracle_threads(), sample="the first round of the same sequences"))


def measure_dssd_round_multi(peaks: dict, src: str, S: int = 32, k: int = 8, K: int = 3, rounds: int = 30) -> dict:
    """Whole DSSD rounds with K draft heads (per position the first confident head supplies the token) on the c1
    shape, the library's table model standing in for the transformer (one table per drafting layer, the shallower
    the noisier); reports the head usage and the mean exit head while drafting, the statistics of the paper's DSSD
    experiments (values of this stand-in, not of a trained model).  The first round is also run by the oracle."""
    import torch
    import oracle
    import paper_2407_21082_b200 as ee
    spec = gen.CONFIGS["c1"]
    d, V = spec["d"], spec["V"]
    cfg = gen.make_config("c1", seed=0, planted=True, M=4, heads=K + 1)
    planting = gen.make_planting(0, f"c1/planted/d{d}/V{V}", d, V)
    sigmas = np.linspace(1.2, 0.4, K)
    tables = [gen.make_markov_model(10 * i, V, d, planting, sigma=float(sg)) for i, sg in enumerate(sigmas)]
    taus = [float(t) for t in np.linspace(0.5, 1.5, K)]

    def bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    E = [bf16(t["E_draft"]) for t in tables] + [bf16(tables[0]["E_verify"])]
    heads = [dict(gamma=torch.from_numpy(hd["gamma"]).cuda(), beta=torch.from_numpy(hd["beta"]).cuda(), W=bf16(hd["W"]))
             for hd in cfg["heads"]]
    for hd, t in zip(heads[:K], taus):
        hd["tau"] = t
    cap = rounds * (k + 1) + 1
    start = ((np.arange(S, dtype=np.int32) * 1543) % V).astype(np.int32)
    state = dict(last_tok=torch.from_numpy(start).cuda(), out_tok=torch.full((S, cap), -9, dtype=torch.int32, device="cuda"),
                 seq_len=torch.zeros(S, dtype=torch.int32, device="cuda"), finished=torch.zeros(S, dtype=torch.uint8, device="cuda"),
                 stats=torch.zeros(4, dtype=torch.int64, device="cuda"))
    rnd = ee.DssdRound(heads[:K], heads[K], 1e-5, k, -1, ee.TableModel(E[:K], E[K], chained=True), state)
    first = {n: v.clone() for n, v in rnd().items()}
    torch.cuda.synchronize()
    first_len = state["seq_len"].cpu().numpy().copy()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(rounds - 1):
        rnd()
    t1.record()
    torch.cuda.synchronize()
    us = 1e3 * t0.elapsed_time(t1) / (rounds - 1)
    status = ee.ee_query_async_error(rnd.workspace)
    stats = state["stats"].cpu().numpy().tolist()
    use = rnd.head_use.cpu().numpy().astype(np.int64)
    ref_state = (np.full((S, cap), -9, np.int32), np.zeros(S, np.int32), np.zeros(S, np.uint8), np.zeros(4, np.int64))
    ref_use = np.zeros(K, np.int64)
    c0 = time.perf_counter()
    ref = oracle.dssd_round_multi([t["E_draft"] for t in tables], tables[0]["E_verify"], cfg["heads"][:K], cfg["heads"][K], taus, -1, k,
                                  start.copy(), *ref_state, ref_use)
    cpu_s = time.perf_counter() - c0
    clean = np.ones(S, bool)
    for c in ref["steps"]:
        for o in c["per_head"]:
            kp = oracle.decisive_rows(o, 1e-3, 1e-3)
            clean[o["rows"][~(kp["argmax"] & kp["exit_mask"])]] = False
    clean &= oracle.decisive_rows(ref["verify_out"], 1e-3, 1e-3)["argmax"].reshape(S, k + 1).all(axis=1)
    agree = bool((first["accept_len"].cpu().numpy()[clean] == ref["accept_len"][clean]).all() and (first_len[clean] == ref_state[1][clean]).all())
    w_bytes = (k * K + 1) * 2.0 * V * d                                   # the heads' weights, once per evaluation
    gbs = w_bytes / (us * 1e-6) / 1e9
    return dict(S=S, k=k, draft_heads=K, taus=taus, d=d, V=V, rounds=rounds, us_per_round=round(us, 1), head_evaluations_per_round=k * K + 1,
                head_use=use.tolist(), mean_exit_head_while_drafting=round(float((np.arange(K) * use).sum() / max(use.sum(), 1)), 3),
                tokens_committed_per_round_per_sequence=round(stats[2] / (rounds * S), 3),
                acceptance_rate=round(stats[1] / max(stats[0], 1), 4), wasted_tokens=stats[0] - stats[1], async_error=status,
                first_round_matches_oracle_on_decisive_sequences=agree, decisive_sequences=int(clean.sum()),
                roofline=dict(bound="hbm", algorithmic_bytes=w_bytes, achieved=round(gbs, 1), peak=peaks["hbm_gbs"], unit="GB/s",
                              frac=round(gbs / peaks["hbm_gbs"], 4), peak_source=f"of {src}", traffic=None,
                              note="K draft heads per drafting step in one launch sequence; the stand-in model is the library's table "
                                   "lookup, launched in the programmatic chain (one small kernel per layer and step)"),
                cpu_baseline=dict(value=float(ref_state[3][2]) / cpu_s, unit="committed tokens/s", seconds=round(cpu_s, 2), kind="oracle",
                                  cores=oracle_threads(), sample="the first round of the same sequences"))


def measure_kl(peaks: dict, src: str, M: int, calls: int = 100) -> dict:
    """ee_head_kl on the c1 shape (one head against the teacher head, M tokens); two copies of both weight
    matrices in rotation (cold L2); the oracle on a sample of the rows."""
    import torch
    import oracle
    import paper_2407_21082_b200 as ee
    cfg = gen.make_config("c1", seed=0, planted=True, M=M, heads=2)
    d, V = cfg["d"], cfg["V"]
    rng = np.random.default_rng(0)
    h_t = gen.bf16_bits_from_f32(gen.f32_from_bf16_bits(cfg["h"]) + rng.normal(0, 0.5, cfg["h"].shape).astype(np.float32))

    def bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    ws = torch.empty(ee.ee_head_kl_workspace_bytes(M, d, V), dtype=torch.uint8, device="cuda")
    ee.ee_workspace_init(ws)
    hh, ht = bf16(cfg["h"]), bf16(h_t)
    prepared = []
    for c in range(2):
        sides = [dict(h=h, gamma=torch.from_numpy(hd["gamma"]).cuda(), beta=torch.from_numpy(hd["beta"]).cuda(), W=bf16(hd["W"]))
                 for h, hd in zip((hh, ht), cfg["heads"])]
        prepared.append(ee.prepare_head_kl(sides[0], sides[1], 1e-5, workspace=ws))
    calls = max(10, calls if M <= 256 else calls // 5)
    for i in range(4):
        prepared[i % 2]()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record()
    for i in range(calls):
        prepared[i % 2]()
    t1.record()
    torch.cuda.synchronize()
    us = 1e3 * t0.elapsed_time(t1) / calls
    got = prepared[(calls - 1) % 2].out["kl"].cpu().numpy()
    rows = min(M, 32)
    c0 = time.perf_counter()
    ref = oracle.kl_to_teacher(cfg["h"][:rows], cfg["heads"][0], h_t[:rows], cfg["heads"][1])
    cpu_s = time.perf_counter() - c0
    nbytes = 2 * (2.0 * V * d + 2.0 * M * d) + 4.0 * M
    flops = 2 * 2.0 * M * V * d
    gbs, tfs = nbytes / (us * 1e-6) / 1e9, flops / (us * 1e-6) / 1e12
    hbm_bound = nbytes / (peaks["hbm_gbs"] * 1e9) >= flops / (peaks["bf16_tflops"] * 1e12)
    roof = (dict(bound="hbm", achieved=round(gbs, 1), peak=peaks["hbm_gbs"], unit="GB/s", frac=round(gbs / peaks["hbm_gbs"], 4)) if hbm_bound
            else dict(bound="tensor", achieved=round(tfs, 1), peak=peaks["bf16_tflops"], unit="TFLOP/s", frac=round(tfs / peaks["bf16_tflops"], 4)))
    roof.update(peak_source=f"of {src}", traffic=None, algorithmic_bytes=nbytes, flops=flops)
    if not hbm_bound:
        roof.update(peak_source=f"of {src} (burst)", frac_of_sustained=round(tfs / peaks["bf16_tflops_sustained"], 4))
    return dict(M=M, d=d, V=V, us_per_call=round(us, 2), launches=3, tokens_per_s=M / (us * 1e-6), roofline=roof,
                max_abs_error_vs_oracle=float(np.abs(got[:rows] - ref["kl"]).max()), loss=float(prepared[(calls - 1) % 2].out["loss"][0].item()),
                cpu_baseline=dict(value=rows / cpu_s, unit="tokens/s", seconds=round(cpu_s, 2), kind="oracle", cores=oracle_threads(),
                                  sample=f"the first {rows} tokens"))


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count() or 1


def oracle_step(cfg: dict, rows: int, heads: int, keep: list | None = None):
    """The oracle's version of a step on the first `rows` rows and `heads` heads.  Returns rows*heads."""
    import oracle
    hb = cfg["h_draft" if "h_draft" in cfg else "h"][:rows]
    tau = cfg["tau_per_row"][:rows] if "tau_per_row" in cfg else cfg["tau"]
    outs = []
    for k, hd in enumerate(cfg["heads"][:heads]):
        hk = cfg["h_verify"][:rows] if ("h_verify" in cfg and k > 0) else hb      # the verify head reads its own rows
        outs.append(oracle.exit_head(hk, hd["gamma"], hd["beta"], hd["ln_eps"], hd["W"], tau))
    if keep is not None:
        keep.extend(outs)
    oracle.compact(outs[0]["exit_mask"], hb)
    S = rows // 8
    if S:
        oracle.dssd_accept(outs[0]["argmax"][:S * 8].reshape(S, 8), outs[0]["exit_mask"][:S * 8].reshape(S, 8),
                           outs[-1]["argmax"][:S * 8].reshape(S, 8))
    return rows * heads


def parity_report(gpu_outs: list, ref_outs: list) -> dict:
    """The timed workload's device results against the oracle's on the rows the oracle evaluated."""
    import oracle
    rep = dict(rows=int(ref_outs[0]["entropy"].size), heads=len(ref_outs), max_abs_dH=0.0, max_abs_dP=0.0,
               argmax_mismatch=0, mask_mismatch=0, excluded_argmax=0, excluded_mask=0, exit_fraction=0.0)
    for got, ref in zip(gpu_outs, ref_outs):
        n = ref["entropy"].size
        keep = oracle.decisive_rows(ref, 1e-3, 1e-3)
        g = {k: v[:n] for k, v in got.items()}
        rep["max_abs_dH"] = max(rep["max_abs_dH"], float(np.abs(g["entropy"].astype(np.float64) - ref["entropy"]).max()))
        rep["max_abs_dP"] = max(rep["max_abs_dP"], float(np.abs(g["maxprob"].astype(np.float64) - ref["maxprob"]).max()))
        rep["argmax_mismatch"] += int(((g["argmax"] != ref["argmax"]) & keep["argmax"]).sum())
        rep["mask_mismatch"] += int(((g["exit_mask"] != ref["exit_mask"]) & keep["exit_mask"]).sum())
        rep["excluded_argmax"] += int((~keep["argmax"]).sum())
        rep["excluded_mask"] += int((~keep["exit_mask"]).sum())
        rep["exit_fraction"] += float(ref["exit_mask"].mean()) / len(ref_outs)
    rep["tolerance"] = "entropy, maxprob within 2e-3; argmax / mask exact outside top-2 gap < 1e-3 and |H - tau| < 1e-3"
    return rep


def cpu_baseline(cfg: dict, steps: int = 1, warmup: int = 0, keep: list | None = None) -> dict:
    """Times the oracle, as it stands, on the host cores on a bounded sample of the headline workload.  The oracle
    decodes a head's bf16 weights to fp64 inside every call; what share of the time that is, is timed separately
    and reported, so that the figure can be read either way."""
    import oracle
    rows, heads = min(cfg["M"], 64), len(cfg["heads"])
    for _ in range(warmup):
        oracle_step(cfg, rows, heads)
    t0 = time.perf_counter()
    done = 0
    for i in range(steps):
        done += oracle_step(cfg, rows, heads, keep if i == 0 else None)
    dt = time.perf_counter() - t0
    t1 = time.perf_counter()
    for hd in cfg["heads"][:heads]:
        oracle.bf16_decode(hd["W"]).T.copy()
    decode = (time.perf_counter() - t1) * steps
    share = min(1.0, decode / dt) if dt > 0 else 0.0
    return dict(value=done / dt, unit=UNIT, cores=oracle_threads(), kind="oracle", seconds=round(dt, 2),
                weight_decode_share=round(share, 3), value_without_weight_decode=done / max(dt - decode, 1e-9),
                sample=f"{steps} step(s) of all {rows} rows x {heads} heads of the workload (fp64 numpy; the oracle decodes "
                       f"each head's weights from bf16 per call, {100 * share:.0f} % of the time here)")


# --------------------------------------------------------------------------------------------- main


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat the timed regions until about this much device time is spent on each (0: one region, for profiler runs)")
    ap.add_argument("--workload", default="c1")
    ap.add_argument("--rows", type=int, default=None, help="override M of the workload")
    ap.add_argument("--path", default="auto", choices=["auto", "stream", "tcgen05", "skinny"], help="force a kernel")
    ap.add_argument("--sweep", action="store_true", help="time every kernel that accepts the size, for c1 at several M")
    ap.add_argument("--no-extra", action="store_true", help="skip the per-config table and the CPU baseline")
    ap.add_argument("--only", default=None, choices=["calibration", "cascade", "dssd_round", "dssd_round_multi", "kl_loss", "read_stream"],
                    help="run that entry of the table alone and print its JSON (for profiling one kernel family)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    spec = gen.CONFIGS[args.workload]
    M = args.rows if args.rows is not None else spec["M"]
    config = dict(workload=f"{args.workload}: Pythia-shaped exit heads d={spec['d']} V={spec['V']} M={M} heads={spec['heads']}",
                  rows_per_gpu=M, heads=spec["heads"], d=spec["d"], V=spec["V"], seed=0,
                  step="ee_exit_head_multi on the batch, then ee_compact_accept: compaction of head 0's survivors + dssd_accept(head 0 vs last head, k=8)")

    if args.impl == "reference":
        if rank != 0:
            return
        cfg = gen.make_config(args.workload, seed=0, planted=False, M=M)
        steps = max(1, min(args.steps, 3))
        base = cpu_baseline(cfg, steps=steps, warmup=min(args.warmup, 1))
        config["l2"] = "n/a (CPU)"
        line = dict(metric=METRIC, value=base["value"], unit=UNIT, n_gpus=args.gpus, steps=steps, warmup=min(args.warmup, 1),
                    ms_per_step=1e3 * base["seconds"] / steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="f64", data="synthetic", config=config, impl="reference", cpu_baseline=base,
                    e2e=dict(value=base["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
        print(json.dumps(line))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ):   # under torchrun, also with one rank
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks, peak_src = load_peaks()
    if args.only is not None:
        if rank == 0:
            rows = [args.rows] if args.rows is not None else [64, 4096]
            entry = {"calibration": lambda: measure_calibration(peaks, peak_src),
                     "cascade": lambda: measure_cascade(peaks, peak_src, M=args.rows or 64),
                     "dssd_round": lambda: measure_dssd_round(peaks, peak_src),
                     "dssd_round_multi": lambda: measure_dssd_round_multi(peaks, peak_src),
                     "read_stream": lambda: measure_read_stream(peaks, peak_src),
                     "kl_loss": lambda: [measure_kl(peaks, peak_src, m) for m in rows]}[args.only]()
            print(json.dumps({args.only: entry}))
        if dist is not None:
            dist.destroy_process_group()
        return

    n_copies = {"c0": 8, "c1": 2}.get(args.workload, 2)
    path = dict(auto=0, stream=1, tcgen05=2, skinny=3)[args.path]
    from paper_2407_21082_b200 import replicas
    wl = Workload(args.workload, M, seed=replicas.rank_seed(0, rank), n_copies=n_copies, path=path)
    config["kernel"] = args.path
    sampler = ClockSampler(local_rank) if rank == 0 else None
    res = measure(wl, args.steps, args.warmup, dist, sampler, min_seconds=args.min_seconds)
    n_heads = len(wl.heads)
    value = res["units_per_s"]                       # head evaluations of all ranks / time of the slowest rank
    config["l2"] = (f"inputs larger than L2: the step cycles through {wl.w_bytes_total / 1e6:.0f} MB of head weights "
                    f"({n_heads} heads x {n_copies} copies) against a 126 MB L2")
    config["parallelism"] = f"replicas x{world} (independent batches, no collective)"
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=res["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic", config=config, clocks=res["clocks"],
                gpu_launches=wl.launches_per_step * args.steps,          # per timed region of `steps` steps
                head_call_us=res["head_call_us"], head_call_us_inner_events=res["head_call_us_inner_events"],
                tail_us=res["tail_us"], repeats=res["repeats"],
                timing=dict(region="`steps` consecutive steps between two CUDA events, barrier and synchronise on both sides",
                            repeats=res["repeats"], reported="median over the repeats (max over ranks per repeat)",
                            ms_per_step_first_repeat=res["ms_per_step_first_repeat"], ms_per_step_min=res["ms_per_step_min"],
                            ms_per_step_max=res["ms_per_step_max"], head_call_us_first_repeat=res["head_call_us_first_repeat"]))
    line["roofline"] = roofline(wl, res["head_call_us"], peaks, peak_src)
    traffic, traffic_note = measured_traffic(wl)
    heads_per_launch = n_heads if wl.multi else 1
    line["roofline"].update(traffic=traffic, traffic_note=traffic_note,
                            launch=dict(heads=heads_per_launch, algorithmic_bytes=heads_per_launch * wl.bytes_per_call,
                                        flops=heads_per_launch * wl.flops_per_call,
                                        us=heads_per_launch * res["head_call_us"]))
    line["roofline"]["kernel"] = (("ee_exit_head_plan_run: %d head(s) in one launch sequence; " % n_heads if wl.multi else
                                   "one ee_exit_head call (%d launch(es)); " % wl.head_launches) +
                                  "duration = CUDA events around `steps` consecutive head evaluations (no event between launches: "
                                  "one would break their programmatic dependent launch chain), averaged per head; "
                                  "tail_us = step time minus that")
    config["heads_call"] = ("ee_exit_head_plan_run (plan of all heads, initialised once)" if wl.multi else "ee_exit_head_path per head")
    gpu_outs = [{k: v.cpu().numpy() for k, v in o.items()} for o in wl.outs] if rank == 0 else None
    if rank == 0:
        line["e2e"] = measure_e2e(wl, max(10, args.steps // 4), 3)
        if world > 1:
            line["e2e"]["note"] = "rank 0 only"
    if not args.no_extra and rank == 0 and world == 1:
        extra = {}
        del wl
        torch.cuda.empty_cache()
        table = [("c0", None, 8, 200), ("c1", 1, 2, 200), ("c1", 4, 2, 200), ("c1", 16, 2, 200), ("c1", 64, 2, 200),
                 ("c2", None, 2, 100), ("c3", None, 2, 100), ("c4", None, 2, 10)]
        per_config = {}
        for name, rows, copies, steps in table:
            w = Workload(name, rows, seed=0, n_copies=copies)
            r = measure(w, steps, 5, min_seconds=0.4)
            key = name if rows is None else f"{name}_M{rows}"
            roof = roofline(w, r["head_call_us"], peaks, peak_src)
            roof["traffic"], roof["traffic_note"] = measured_traffic(w)      # per launch, like the headline's
            extra[key] = dict(M=w.M, d=w.d, heads=len(w.heads), head_call_us=round(r["head_call_us"], 2),
                              head_call_us_first_repeat=round(r["head_call_us_first_repeat"], 2), repeats=r["repeats"],
                              tail_us=round(r["tail_us"], 2), tokens_per_s=w.M / (r["head_call_us"] * 1e-6),
                              roofline=roof, launches_per_head=w.head_launches)
            # the same figures in short, inside the roofline object of the line
            short = dict(us=round(r["head_call_us"], 2), bound=roof["bound"], frac=roof["frac"], achieved=roof["achieved"],
                         unit=roof["unit"], traffic=roof["traffic"], tokens_per_s=round(w.M / (r["head_call_us"] * 1e-6), 1),
                         repeats=r["repeats"], steps_per_repeat=steps)
            for extra_key in ("tensor_frac", "hbm_frac", "frac_of_sustained"):
                if extra_key in roof:
                    short[extra_key] = roof[extra_key]
            per_config[key] = short
            del w
            torch.cuda.empty_cache()
        line["roofline"]["per_config"] = per_config
        line["roofline"]["per_config_note"] = ("us = one head evaluation (median over the repeats of a region of steps_per_repeat "
                                               "consecutive head evaluations, at least 0.4 s in all), frac against the bound named")
        line["configs"] = extra
        line["roofline"]["read_stream"] = measure_read_stream(peaks, peak_src)
        line["calibration"] = measure_calibration(peaks, peak_src)
        line["cascade"] = measure_cascade(peaks, peak_src)
        line["dssd_round"] = measure_dssd_round(peaks, peak_src)
        line["dssd_round_multi"] = measure_dssd_round_multi(peaks, peak_src)
        line["kl_loss"] = [measure_kl(peaks, peak_src, M) for M in (64, 4096)]
        if args.sweep:
            sweep = {}
            for rows in (1, 8, 16, 32, 64):
                for mk in ("stream", "skinny", "gemm"):
                    os.environ["EE_MULTI_KERNEL"] = mk
                    w = Workload("c1", rows, seed=0, n_copies=2)
                    sweep[f"c1_M{rows}_multi_{mk}"] = round(measure(w, 300, 5)["head_call_us"], 2)
                    del w
                    torch.cuda.empty_cache()
                os.environ.pop("EE_MULTI_KERNEL", None)
                for pname, pid in (("stream", 1), ("skinny", 3), ("tcgen05", 2)):
                    w = Workload("c1", rows, seed=0, n_copies=2, path=pid, multi=False)
                    if w.head_launches == 0:
                        continue
                    r = measure(w, 300, 5)
                    sweep[f"c1_M{rows}_{pname}"] = round(r["head_call_us"], 2)
                    del w
                    torch.cuda.empty_cache()
            line["sweep_head_call_us"] = sweep
        cfg = gen.make_config(args.workload, seed=0, planted=False, M=M)
        ref_outs = []
        line["cpu_baseline"] = cpu_baseline(cfg, steps=6, warmup=0, keep=ref_outs)   # about ten seconds of host work
        line["parity"] = parity_report(gpu_outs, ref_outs)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
