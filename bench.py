#!/usr/bin/env python
"""Benchmark of the batched LoRA-delta hot path on B200.

One step = one pass of the whole hot path over one batch: bucket the batch's
adapter ids once, then apply the LoRA delta of every (layer, projection) pool
of the workload (for the default decode workload: 32 layers x q/k/v/o = 128
calls over a 33.6 GB pool of 1000 rank-16 adapters per projection).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--config 2|3|4|5|6] [--layers L] [--graph 0|1] [--tp]

Prints ONE JSON line (rank 0).  `value` is tokens per second through the whole
step with inputs resident in HBM; `e2e` is the same step through the host-buffer
entry point (pinned host memory, copies inside the timed region); `roofline`
compares the dominant kernel's algorithmic bytes per launch with the measured
HBM copy bandwidth and with a read-only streaming bandwidth measured in the same
run; `cpu_baseline` is the float64 oracle timed on this machine's host cores on a
bounded sample.  The step's x, ids and y are resident before the step starts, and the
benchmark says so to the library (plora_set_inputs_resident; --resident 0 withholds
the hint): the fused kernels then read x while the previous launch drains.
`roofline.frac_without_inputs_hint` is the same set of launches without the hint.
Without --config the headline (config 2) is followed, in the
same process, by the other benchmark workloads (configs 3 to 6 and decode
attention), each with its own roofline, full-size parity figure, oracle time and
clocks, under the key `per_config`.  --impl reference times the oracle alone.
--gpus N without a launcher's environment starts N ranks itself (one process per
GPU: replicas of the step, or with --tp the tensor-parallel adapter wave).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from workloads import gen_pool_device, make_workload  # noqa: E402

FALLBACK_HBM_GBS = 6650.0   # used only when MEASURED_PEAKS.json is absent

# DRAM bytes (read + write) per (layer, proj) delta of the dominant kernel, from ncu captures of this
# library; the roofline entry scales the figure to the average launch (a launch may carry a group of
# projections).  A capture says nothing about a later build of the kernels: the line prints the commit the
# kernels of the capture were built from next to the figure, and null for a workload that was not captured.
NCU_TRAFFIC_BUILD = "a5cdd72"          # the tensor-core kernels, the one-rank kernels of the mixed workload, attention
NCU_TRAFFIC_BUILD_LAZY = "c047e8b"     # the fused kernels that join the stream order late (the decode workloads)
NCU_TRAFFIC_BUILD_SKEW = "ce7d1ff"     # the all-classes kernel with its final task plan
NCU_TRAFFIC_BYTES = {
    "decode7b": 40.4e6,    # q/k/v launch 122.19 / 120.63 MB, o launch 40.30 / 40.35 MB, over four projections
    # captured with 150 adapters per pool (2106.4 MB of traffic for 2116.3 MB of algorithmic bytes over one layer's
    # four launches); the full workload's algorithmic bytes are scaled by this ratio
    "decode13b": ("of_algorithmic", 2106.4 / 2116.3),
    "prefill": 622.2e6,    # the wide tensor-core kernel, one projection
    "mixed": 525.7e6,      # the four rank-class launches and the split tensor-core launch of one projection
    "skew7b": 93.5e6,      # q/k/v launch 277.62 MB, o launch 96.26 MB, over four projections
}
NCU_TRAFFIC_LAZY = ("decode7b", "decode13b", "skew7b")
# decode attention, per call (one layer's cache) of the partial kernel, at the default shapes with one query head per KV head
NCU_ATTN_TRAFFIC_BYTES = {False: 2604.8e6, True: 3241.3e6}   # short requests / long requests


# ----------------------------------------------------------------------------------
# accounting (the paper's cost model, Section VI-B: the memory term of strategy E1
# counts every adapter present once, 2 bytes per value; generalised to d_in != d_out)
# ----------------------------------------------------------------------------------
def algorithmic_bytes(ids: np.ndarray, ranks: np.ndarray, d_in: int, d_out: int) -> dict:
    act = ids[ids >= 0]
    distinct = np.unique(act)
    adapter = int(sum((d_in + d_out) * int(ranks[a]) * 2 for a in distinct))
    x_bytes = int(len(ids) * d_in * 2)
    y_bytes = int(len(act) * d_out * 8)   # fp32 read + write
    return dict(adapter=adapter, x=x_bytes, y=y_bytes, total=adapter + x_bytes + y_bytes, distinct=int(len(distinct)))


def algorithmic_flops(ids: np.ndarray, ranks: np.ndarray, d_in: int, d_out: int) -> int:
    act = ids[ids >= 0]
    return int(2 * sum(int(ranks[a]) for a in act) * (d_in + d_out))


def hbm_floor_ms(n_bytes: float, gbs: float) -> float:
    return n_bytes / (gbs * 1e9) * 1e3


def measured_peaks() -> dict:
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, source="fallback")


# ----------------------------------------------------------------------------------
# clocks sampling during the timed region
# ----------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            c = [v.strip() for v in r.split(",")]
            if len(c) < 7:
                continue
            try:
                sm.append(float(c[0])); mx.append(float(c[1]))
            except ValueError:
                continue
            for n, v in zip(names, c[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


# ----------------------------------------------------------------------------------
# workload set-up on the device
# ----------------------------------------------------------------------------------
class DeviceWorkload:
    """Pools registered in a library context plus per-call activations, all resident in HBM."""

    def __init__(self, wl, device_index: int, max_tokens=None, fp16: bool = False, resident: bool = True):
        import torch
        import paper_2608_05483_b200 as P
        self.P, self.torch, self.wl = P, torch, wl
        self.dev = f"cuda:{device_index}"
        torch.cuda.set_device(device_index)
        self.fp16 = fp16
        self.ctx = P.Context(max_tokens or wl.n_tok, wl.n_adapters, device=device_index)
        if fp16:
            self.ctx.set_input_type(True)
        # every x of the step sits in HBM before the step starts: the kernels may read it while the previous one drains
        self.ctx.set_inputs_resident(resident)
        self.ids = torch.from_numpy(wl.ids).to(self.dev)
        g = torch.Generator(device=self.dev)
        g.manual_seed(wl.seed)
        self.x = {}
        self.y = {}
        self.grouped = True
        self._groups = None
        for pool in wl.pools:
            A, B = gen_pool_device(wl, pool, self.dev, fp16)
            self.ctx.register_pool(pool.layer, pool.proj, pool.d_in, pool.d_out, wl.ranks, wl.scales, A, B)
            del A, B
            key = (pool.layer, pool.x_group)
            if key not in self.x:
                self.x[key] = torch.randn((wl.n_tok, pool.d_in), generator=g, device=self.dev,
                                          dtype=torch.float32).to(torch.float16 if fp16 else torch.bfloat16)
            self.y[(pool.layer, pool.proj)] = torch.randn((wl.n_tok, pool.d_out), generator=g, device=self.dev,
                                                          dtype=torch.float32)
        torch.cuda.synchronize()

    def groups(self):
        """The calls of one step: projections of a layer that do not depend on one another go
        together (q/k/v read the same activations, so do up/gate); o and down stand alone."""
        if self._groups is None:
            by = {}
            for pool in self.wl.pools:
                by.setdefault((pool.layer, pool.x_group), []).append(pool)
            self._groups = [by[k] for k in sorted(by)]
        return self._groups

    def deltas(self):
        """Every (layer, proj) delta of the step; enqueue only."""
        ctx = self.ctx
        for grp in self.groups():
            if self.grouped and len(grp) > 1:
                ctx.lora_delta_group([self.x[(p.layer, p.x_group)] for p in grp], self.ids, [p.layer for p in grp],
                                     [p.proj for p in grp], [self.y[(p.layer, p.proj)] for p in grp])
            else:
                for p in grp:
                    ctx.lora_delta(self.x[(p.layer, p.x_group)], self.ids, p.layer, p.proj, self.y[(p.layer, p.proj)])

    def step(self):
        """bucket once, then every (layer, proj) delta; enqueue only."""
        self.ctx.bucket(self.ids, self.wl.n_adapters)
        self.deltas()

    def host_adapters(self, pool, adapters):
        """Logical A/B bit patterns of `adapters` of `pool`, regenerated on the device and copied to the host."""
        A, B = gen_pool_device(self.wl, pool, self.dev, self.fp16)
        outA = [None] * self.wl.n_adapters
        outB = [None] * self.wl.n_adapters
        for a in adapters:
            outA[int(a)] = A[int(a)].contiguous().view(self.torch.int16).cpu().numpy().view(np.uint16)
            outB[int(a)] = B[int(a)].contiguous().view(self.torch.int16).cpu().numpy().view(np.uint16)
        return outA, outB

    def close(self):
        self.ctx.close()


def bits_of(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


# ----------------------------------------------------------------------------------
# the CPU oracle on a bounded sample (also a full-size parity check of sampled pools)
# ----------------------------------------------------------------------------------
def oracle_sample(dw: DeviceWorkload, n_pools: int, check_gpu: bool, target_s: float = 0.0, pools=None):
    import oracle
    oracle.set_input_type(dw.fp16)
    try:
        return _oracle_sample(dw, n_pools, check_gpu, target_s, pools)
    finally:
        oracle.set_input_type(False)


def _oracle_sample(dw: DeviceWorkload, n_pools: int, check_gpu: bool, target_s: float = 0.0, pools=None):
    """Times the oracle on `n_pools` (layer, proj) calls of the step at full size.  When one pass
    over them takes less than `target_s`, every call is repeated (same inputs) so that the whole
    sample is about `target_s` of CPU work; returns the time of ONE pass (the mean)."""
    import oracle
    wl = dw.wl
    torch = dw.torch
    if pools is None:
        pools = wl.pools[:: max(1, len(wl.pools) // n_pools)][:n_pools]
    distinct = wl.distinct_adapters()
    cpu_s, max_err, repeats = 0.0, 0.0, 1
    for i, pool in enumerate(pools):
        A, B = dw.host_adapters(pool, distinct)
        x = bits_of(dw.x[(pool.layer, pool.x_group)])
        y_in = dw.y[(pool.layer, pool.proj)].cpu().numpy().copy()
        t0 = time.perf_counter()
        ref = oracle.lora_delta(x, wl.ids, wl.ranks, wl.scales, A, B, pool.d_out, y_in)
        first = time.perf_counter() - t0
        if i == 0 and target_s > 0:
            repeats = int(max(1, min(200, round(target_s / max(first * len(pools), 1e-6)))))
        t0 = time.perf_counter()
        for _ in range(repeats - 1):
            oracle.lora_delta(x, wl.ids, wl.ranks, wl.scales, A, B, pool.d_out, y_in)
        cpu_s += (first + time.perf_counter() - t0) / repeats
        if check_gpu:
            # through the call the timed step makes for this pool: with its group when calls are grouped
            grp = next(g for g in dw.groups() if pool in g)
            ys = {(q.layer, q.proj): dw.y[(q.layer, q.proj)].clone() for q in grp}
            if dw.grouped and len(grp) > 1:
                dw.ctx.lora_delta_group([dw.x[(q.layer, q.x_group)] for q in grp], dw.ids, [q.layer for q in grp],
                                        [q.proj for q in grp], [ys[(q.layer, q.proj)] for q in grp])
            else:
                dw.ctx.lora_delta(dw.x[(pool.layer, pool.x_group)], dw.ids, pool.layer, pool.proj, ys[(pool.layer, pool.proj)])
            y = ys[(pool.layer, pool.proj)]
            torch.cuda.synchronize()
            delta_scale = float(np.max(np.abs(ref - y_in)))
            max_err = max(max_err, float(np.max(np.abs(y.cpu().numpy() - ref)) / delta_scale))
    return pools, cpu_s, max_err, oracle.threads(), repeats


# ----------------------------------------------------------------------------------
# replicas: every rank runs its own batch on its own GPU; the only thing that crosses ranks is
# the timing (max over ranks), never data of the path
# ----------------------------------------------------------------------------------
def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks (the value itself when no process group is up)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(n_tok_per_rank: int, world: int, ms_per_step_max: float) -> float:
    """Weak scaling: the job processed world * n_tok tokens in the slowest rank's step time."""
    return world * n_tok_per_rank / (ms_per_step_max * 1e-3)


# ----------------------------------------------------------------------------------
# read-only streaming bandwidth, measured in this run with the library's probe kernel
# ----------------------------------------------------------------------------------
_READ_PEAK = {}


def measured_read_gbs(device_index: int) -> float:
    """GB/s of a kernel that only reads (16-byte loads over a 4 GiB buffer, far larger than L2): best of 10
    launches after 3 warm-ups, CUDA events.  The decode kernels' traffic is almost all reads, so this is the
    ceiling they can be held against; the copy figure in MEASURED_PEAKS.json counts reads and writes."""
    if device_index in _READ_PEAK:
        return _READ_PEAK[device_index]
    import torch
    import paper_2608_05483_b200 as P
    dev = f"cuda:{device_index}"
    n = 4 << 30
    buf = torch.empty(n, dtype=torch.uint8, device=dev)
    buf.view(torch.int32).fill_(0x01010101)
    sink = torch.zeros(1 << 16, dtype=torch.uint8, device=dev)
    st = int(torch.cuda.current_stream().cuda_stream)
    best = float("inf")
    for i in range(13):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rc = P.plora_stream_read(buf.data_ptr(), n, sink.data_ptr(), int(sink.numel()), st)
        e1.record()
        torch.cuda.synchronize()
        if rc != 0:
            raise RuntimeError(f"plora_stream_read: {rc}")
        if i >= 3:
            best = min(best, e0.elapsed_time(e1))
    del buf, sink
    torch.cuda.empty_cache()
    _READ_PEAK[device_index] = n / (best * 1e-3) / 1e9
    return _READ_PEAK[device_index]


def shared_x_bytes(wl, groups) -> int:
    """Algorithmic bytes of a step when projections that go into one launch read their common x once."""
    total = 0
    for grp in groups:
        per = [algorithmic_bytes(wl.ids, wl.ranks, p.d_in, p.d_out) for p in grp]
        total += sum(b["adapter"] + b["y"] for b in per) + per[0]["x"]
    return total


def parity_pools(wl):
    """One pool per distinct projection shape (the first of each): what the full-size parity check covers."""
    seen, out = set(), []
    for p in wl.pools:
        if (p.d_in, p.d_out) not in seen:
            seen.add((p.d_in, p.d_out))
            out.append(p)
    return out


# ----------------------------------------------------------------------------------
# one workload, measured
# ----------------------------------------------------------------------------------
def measure_lora(cfg: int, args, local: int, world: int, rank: int, headline: bool) -> dict:
    """Times workload `cfg` on this rank's GPU and returns the pieces of the result line.  headline: the
    full protocol (all sampled pools for the oracle, the end-to-end leg); otherwise the shorter one of a
    `per_config` entry (whole-output parity on one pool per projection shape, a few seconds of oracle time)."""
    import torch
    import torch.distributed as dist
    import paper_2608_05483_b200 as P

    wl = make_workload(cfg, n_layers=args.layers if headline else None, n_adapters=args.adapters if headline else None)
    dw = DeviceWorkload(wl, local, fp16=args.dtype == "fp16", resident=bool(args.resident))
    dw.grouped = not args.no_group
    ctx = dw.ctx
    ctx.set_path({"auto": P.PATH_AUTO, "fused": P.PATH_FUSED, "unfused": P.PATH_UNFUSED, "sgmv": P.PATH_SGMV,
                  "sgmv_split": P.PATH_SGMV_SPLIT}[args.path])
    n_calls = len(wl.pools)
    steps = args.steps if headline else max(10, min(args.steps, 50))
    warmup = max(3, args.warmup)

    # full-size parity + the oracle's time, before anything is timed (rank 0)
    cpu = None
    parity = None
    if rank == 0 and not args.no_cpu:
        if headline:
            pools, cpu_s, parity, threads, repeats = oracle_sample(dw, args.cpu_pools, check_gpu=True,
                                                                   target_s=args.cpu_seconds)
        else:
            pools, cpu_s, parity, threads, repeats = oracle_sample(dw, 0, check_gpu=True, target_s=args.cpu_seconds / 5,
                                                                   pools=parity_pools(wl))
        # scale the sampled calls to the whole step by algorithmic flops (the pools of a step differ in shape)
        fl = lambda ps: sum(algorithmic_flops(wl.ids, wl.ranks, p.d_in, p.d_out) for p in ps)
        scaled = cpu_s * fl(wl.pools) / fl(pools)
        cpu = dict(value=wl.n_tok / scaled, unit="tokens/s", cores=threads, kind="oracle",
                   sample=f"{len(pools)} of {n_calls} (layer, proj) calls at full size ({wl.n_tok} tokens, whole output "
                          f"compared with the GPU's), each run {repeats}x: {cpu_s * repeats:.1f} s of oracle time, "
                          f"mean pass scaled to the whole step by flops")

    stream = torch.cuda.current_stream()

    def capture(fn):
        if not args.graph:
            return None, 0
        s = torch.cuda.Stream()
        s.wait_stream(stream)
        with torch.cuda.stream(s):
            fn()
        stream.wait_stream(s)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        lc0 = ctx.launch_count()
        with torch.cuda.graph(g):
            fn()
        return g, ctx.launch_count() - lc0   # kernels recorded in the graph = launched per replay

    graph, launches_per_step = capture(dw.step)

    def one_step():
        graph.replay() if graph is not None else dw.step()

    for _ in range(warmup):
        one_step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    l0 = ctx.launch_count()
    ev[0].record()
    for k in range(steps):
        one_step()
    ev[1].record()
    torch.cuda.synchronize()
    launches = steps * launches_per_step if graph is not None else ctx.launch_count() - l0
    total_ms = ev[0].elapsed_time(ev[1])
    clocks = sampler.stop()
    total_ms = max_over_ranks(total_ms, f"cuda:{local}")
    if world > 1:
        dist.barrier()
    ms_per_step = total_ms / steps

    # kernel-only timing for the roofline: the delta calls of one step without the bucket kernel,
    # replayed from a CUDA graph like the step itself so that host launch cost does not pace them
    ctx.bucket(dw.ids, wl.n_adapters)
    torch.cuda.synchronize()
    kgraph, delta_launches = capture(dw.deltas)
    if kgraph is None:
        lc1 = ctx.launch_count()
        dw.deltas()
        torch.cuda.synchronize()
        delta_launches = ctx.launch_count() - lc1
    for _ in range(3):
        kgraph.replay() if kgraph is not None else dw.deltas()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    reps = max(3, min(steps, 50))
    e0.record()
    for _ in range(reps):
        kgraph.replay() if kgraph is not None else dw.deltas()
    e1.record()
    torch.cuda.synchronize()
    deltas_ms = e0.elapsed_time(e1) / reps                 # all delta launches of one step
    kernel_ms = deltas_ms / n_calls                        # per (layer, proj) delta, however they are grouped

    # the same launches without the inputs-resident hint (every kernel touches x only after the one before it has
    # completed): what a caller gets who cannot make that statement about its x
    deltas_ms_no_hint = None
    if args.resident and not args.no_extras:
        ctx.set_inputs_resident(False)
        g2, _ = capture(dw.deltas)
        for _ in range(3):
            g2.replay() if g2 is not None else dw.deltas()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(reps):
            g2.replay() if g2 is not None else dw.deltas()
        e1.record()
        torch.cuda.synchronize()
        deltas_ms_no_hint = e0.elapsed_time(e1) / reps
        ctx.set_inputs_resident(True)
        del g2

    per_call = [algorithmic_bytes(wl.ids, wl.ranks, p.d_in, p.d_out) for p in wl.pools]
    step_bytes = sum(b["total"] for b in per_call)
    step_adapter_bytes = sum(b["adapter"] for b in per_call)
    step_bytes_shared_x = shared_x_bytes(wl, dw.groups()) if dw.grouped else step_bytes
    peaks = measured_peaks()
    read_gbs = None if args.no_read_peak else measured_read_gbs(local)
    # algorithmic bytes per launch / average launch duration, over the step's delta launches (a launch
    # carries one projection or a group of independent ones): equal to step bytes / their total time
    bytes_per_launch = step_bytes / delta_launches
    launch_us = deltas_ms * 1e3 / delta_launches
    achieved = bytes_per_launch / (launch_us * 1e-6) / 1e9
    achieved_shared = step_bytes_shared_x / (deltas_ms * 1e-3) / 1e9
    traffic = NCU_TRAFFIC_BYTES.get(wl.name) if args.dtype == "bf16" and args.path == "auto" else None
    roofline = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=achieved / peaks["hbm_gbs"],
                    traffic=None if traffic is None else (traffic[1] * bytes_per_launch if isinstance(traffic, tuple)
                                                           else traffic * n_calls / delta_launches),
                    traffic_from_build=None if traffic is None else (NCU_TRAFFIC_BUILD_SKEW if wl.name == "skew7b" else NCU_TRAFFIC_BUILD_LAZY if wl.name in NCU_TRAFFIC_LAZY else NCU_TRAFFIC_BUILD),
                    kernel="sgmv_kernel (tensor-core segmented GEMM)" if wl.name == "prefill" else "bgmv_kernel (fused shrink+expand)",
                    peak_source=peaks["source"], avg_launch_us=launch_us, launches_per_step=delta_launches,
                    per_projection_us=kernel_ms * 1e3, algorithmic_bytes_per_launch=bytes_per_launch,
                    # x counted once per launch that serves several projections (what the kernel has to read)
                    frac_shared_x=achieved_shared / peaks["hbm_gbs"], achieved_shared_x=achieved_shared,
                    # against a kernel that only reads, measured in this run (the copy peak counts reads and writes)
                    read_peak=read_gbs, frac_of_read_peak=None if read_gbs is None else achieved / read_gbs,
                    frac_of_nominal_8tbs=achieved / 8000.0,
                    frac_without_inputs_hint=None if deltas_ms_no_hint is None
                    else step_bytes / (deltas_ms_no_hint * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    adapter_bytes_only_gbs=step_adapter_bytes / n_calls / (kernel_ms * 1e-3) / 1e9,
                    step_gbs=step_bytes / (ms_per_step * 1e-3) / 1e9)
    return dict(wl=wl, dw=dw, ms_per_step=ms_per_step, steps=steps, warmup=warmup, clocks=clocks, launches=int(launches),
                roofline=roofline, cpu=cpu, parity=parity, kernel_ms=kernel_ms, step_bytes=step_bytes, n_calls=n_calls,
                distinct=per_call[0]["distinct"])


def measure_e2e(m: dict, args, local: int, world: int) -> dict:
    """The step through the host-buffer entry point: pinned host memory, copies inside the timed region."""
    import torch
    dw, wl, ctx = m["dw"], m["wl"], m["dw"].ctx
    xh = {k: v.cpu().pin_memory() for k, v in list(dw.x.items())}
    yh = {k: v.cpu().pin_memory() for k, v in list(dw.y.items())}
    idh = dw.ids.cpu().pin_memory()

    def host_step():
        # one queued call per group of projections that share their input; results read at the end
        for grp in dw.groups():
            ctx.lora_delta_host_async(xh[(grp[0].layer, grp[0].x_group)], idh, [p.layer for p in grp],
                                      [p.proj for p in grp], [yh[(p.layer, p.proj)] for p in grp])
        ctx.host_sync()

    host_step()
    torch.cuda.synchronize()
    n_e2e = max(1, min(args.steps, 5))
    t0 = time.perf_counter()
    for _ in range(n_e2e):
        host_step()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / n_e2e
    e2e_s = max_over_ranks(e2e_s, f"cuda:{local}")
    h2d = sum(wl.n_tok * grp[0].d_in * 2 + wl.n_tok * 4 + sum(wl.n_tok * p.d_out * 4 for p in grp) for grp in dw.groups())
    d2h = sum(wl.n_tok * p.d_out * 4 for p in wl.pools)
    return dict(value=world * wl.n_tok / e2e_s, unit="tokens/s", h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                ms_per_step=e2e_s * 1e3, steps=n_e2e, api="plora_lora_delta_host_async per group + plora_host_sync",
                host_link_gbs=max(h2d, d2h) / e2e_s / 1e9)


def config_entry(m: dict, args, cfg: int) -> dict:
    wl = m["wl"]
    return dict(workload=f"config {cfg} ({wl.name})", n_tok=wl.n_tok, n_adapters=wl.n_adapters,
                layers=len({p.layer for p in wl.pools}), calls_per_step=m["n_calls"],
                ranks=sorted({int(r) for r in wl.ranks}), ids=wl.meta.get("ids"), accumulate="fp32", y="fp32",
                distinct_adapters=m["distinct"], path=args.path, cuda_graph=bool(args.graph), grouped_calls=not args.no_group,
                inputs_resident_hint=bool(args.resident),
                l2="inputs larger than L2: a step streams %.2f GB through %d distinct slabs" % (m["step_bytes"] / 1e9, m["n_calls"]))


METRIC = "LoRA-delta tokens/sec at 1000 adapters (whole step: bucket + every layer x projection delta)"


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)

    cfg = args.config or 2
    m = measure_lora(cfg, args, local, world, rank, headline=True)
    wl = m["wl"]
    e2e = None if args.no_e2e else measure_e2e(m, args, local, world)
    status = m["dw"].ctx.device_status()
    m["dw"].close()
    m.pop("dw")
    torch.cuda.empty_cache()

    # the other benchmark workloads, one after the other in this process (one GPU only: at N > 1 the line
    # is the replicas' headline and nothing else)
    per_config = None
    if args.config is None and world == 1 and not args.no_extras:
        per_config = {}
        for c in (3, 4, 5, 6):
            mm = measure_lora(c, args, local, world, rank, headline=False)
            st = mm["dw"].ctx.device_status()
            mm["dw"].close()
            mm.pop("dw")
            torch.cuda.empty_cache()
            w = mm["wl"]
            per_config[f"config{c}"] = dict(
                workload=f"config {c} ({w.name})", ms_per_step=mm["ms_per_step"], steps=mm["steps"], warmup=mm["warmup"],
                value=w.n_tok / (mm["ms_per_step"] * 1e-3), unit="tokens/s", roofline=mm["roofline"],
                parity_max_rel_err=mm["parity"], cpu_baseline=mm["cpu"], clocks=mm["clocks"], gpu_launches=mm["launches"],
                config=config_entry(mm, args, c), device_status=st)
        for long_ctx in (False, True):
            a = attention_entry(args, long_ctx=long_ctx, steps=max(5, min(args.steps, 20)))
            per_config["attention_long" if long_ctx else "attention"] = a

    if rank == 0:
        conf = config_entry(m, args, cfg)
        conf["multi_gpu"] = "replicas: every rank runs its own batch, no data-path collective"
        out = dict(metric=METRIC, value=whole_job_tokens_per_s(wl.n_tok, world, m["ms_per_step"]), unit="tokens/s",
                   n_gpus=world, steps=m["steps"], warmup=m["warmup"], ms_per_step=m["ms_per_step"], higher_is_better=True,
                   scaling="weak", vs_baseline=None, dtype=args.dtype, data="synthetic", config=conf, clocks=m["clocks"],
                   e2e=e2e, gpu_launches=m["launches"], roofline=m["roofline"], cpu_baseline=m["cpu"],
                   tokens_per_s_per_call=wl.n_tok / (m["kernel_ms"] * 1e-3), parity_max_rel_err=m["parity"],
                   device_status=status, per_config=per_config)
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_reference(args):
    """The oracle, as it stands, on the host cores.  A step is the whole workload when K + W such steps fit
    in about two minutes, else a bounded sample of its (layer, proj) calls at full size; the line reports the
    milliseconds that were really timed and says how `value` was scaled from them."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from workloads import gen_adapter, gen_x, gen_y_in
    cfg = args.config or 2
    wl = make_workload(cfg, n_layers=args.layers)
    n_calls = len(wl.pools)
    distinct = wl.distinct_adapters()
    warmup = max(0, args.warmup)

    def host_pool(pool):   # host-generated logical matrices for the adapters the batch touches
        A = [None] * wl.n_adapters
        B = [None] * wl.n_adapters
        for a in distinct:
            A[int(a)], B[int(a)] = gen_adapter(wl, pool, int(a))
        return (pool, gen_x(wl, pool), A, B, gen_y_in(wl, pool))

    data = [host_pool(wl.pools[0])]
    pool, x, A, B, y_in = data[0]
    t0 = time.perf_counter()
    oracle.lora_delta(x, wl.ids, wl.ranks, wl.scales, A, B, pool.d_out, y_in)
    one_call = time.perf_counter() - t0
    budget_s = 120.0 / max(1, args.steps + warmup)                 # oracle time one step may take
    n_sample = int(max(1, min(n_calls, budget_s / max(one_call, 1e-6))))
    picked = wl.pools[:: max(1, n_calls // n_sample)][:n_sample]
    data = [host_pool(p) for p in picked]

    def sample_step():
        for pool, x, A, B, y_in in data:
            oracle.lora_delta(x, wl.ids, wl.ranks, wl.scales, A, B, pool.d_out, y_in)

    for _ in range(warmup):
        sample_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        sample_step()
    timed_s = (time.perf_counter() - t0) / args.steps
    fl = lambda ps: sum(algorithmic_flops(wl.ids, wl.ranks, p.d_in, p.d_out) for p in ps)
    factor = fl(wl.pools) / fl(picked)                              # 1.0 when the whole step was timed
    value = wl.n_tok / (timed_s * factor)
    sample = (f"{len(picked)} of {n_calls} (layer, proj) calls per step at full size ({wl.n_tok} tokens)"
              + ("" if len(picked) == n_calls else ", value scaled to the whole step by flops"))
    out = dict(impl="reference", metric=METRIC, value=value, unit="tokens/s", n_gpus=1, steps=args.steps, warmup=warmup,
               ms_per_step=timed_s * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
               data="synthetic",
               scaled_from=dict(calls_timed_per_step=len(picked), calls_per_step=n_calls, ms_timed_per_step=timed_s * 1e3,
                                whole_step_ms=timed_s * factor * 1e3, factor=factor),
               config=dict(workload=f"config {cfg} ({wl.name})", n_tok=wl.n_tok, n_adapters=wl.n_adapters,
                           layers=len({p.layer for p in wl.pools}), calls_per_step=n_calls,
                           ranks=sorted({int(r) for r in wl.ranks}), ids=wl.meta.get("ids"), accumulate="f64", y="f64",
                           distinct_adapters=int(len(distinct))),
               cpu_baseline=dict(value=value, unit="tokens/s", cores=oracle.threads(), kind="oracle", sample=sample),
               e2e=dict(value=value, unit="tokens/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(out), flush=True)


def attention_entry(args, long_ctx: bool, steps: int) -> dict:
    """Decode attention (the paper's other memory-bound operator) on a synthetic batch: one query token per
    request against a KV cache of the paper's request lengths, Llama-2-7B head shapes (32 heads of 128),
    several layers' caches in turn.  Returns the result as a dict (a line of its own with --op attention, an
    entry of `per_config` otherwise)."""
    import torch
    import paper_2608_05483_b200 as P
    torch.cuda.set_device(0)
    dev = "cuda:0"
    n_req, lo, hi = (64, 2048, 4096) if long_ctx else (256, 100, 1024)
    n_req = args.attn_requests or n_req
    G = args.attn_q_per_kv
    H, d = 32 // G, 128      # KV heads: 32 query heads in all, G of them per KV head
    Hq = H * G
    rng = np.random.default_rng(20260805 * 10 + (8 if long_ctx else 7))
    kv_len = rng.integers(lo, hi + 1, size=n_req).astype(np.int32)
    g = torch.Generator(device=dev)
    g.manual_seed(int(rng.integers(1 << 30)))
    layers = args.attn_layers      # several layers' caches in turn, so that a step streams far more than L2 holds
    q = torch.randn((layers, n_req, Hq, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    K = torch.randn((layers, n_req, H, hi, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    V = torch.randn((layers, n_req, H, hi, d), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    lens = torch.from_numpy(kv_len).to(dev)
    scale = 1.0 / float(np.sqrt(d))
    out = torch.empty((layers, n_req, Hq, d), dtype=torch.float32, device=dev)
    ws = torch.zeros(P.plora_attn_workspace_bytes(n_req, hi, H, G), dtype=torch.uint8, device=dev)

    def step():
        for l in range(layers):
            P.attn_decode(q[l], K[l], V[l], lens, scale, out=out[l], workspace=ws)

    warmup = max(3, args.warmup)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / steps
    rc, status = P.plora_attn_status(ws.data_ptr())
    kv_bytes = float(kv_len.sum()) * H * d * 2 * 2 * layers            # K and V, 2 bytes per value
    other = layers * n_req * Hq * d * (2 + 4)                          # q read, out written
    peaks = measured_peaks()
    read_gbs = None if args.no_read_peak else measured_read_gbs(0)
    achieved = (kv_bytes + other) / (ms * 1e-3) / 1e9
    # parity on sampled requests and the oracle's time on them
    from oracle.attention import decode_attention
    sample = np.unique(np.concatenate([[0, n_req - 1, int(np.argmax(kv_len)), int(np.argmin(kv_len))], rng.integers(0, n_req, size=4)]))
    Ks = K[0][sample].float().cpu().numpy().astype(np.float64)
    Vs = V[0][sample].float().cpu().numpy().astype(np.float64)
    qs = q[0][sample].float().cpu().numpy().astype(np.float64)
    t0 = time.perf_counter()
    ref = decode_attention(qs, Ks, Vs, kv_len[sample], scale)
    cpu_s = time.perf_counter() - t0
    err = float(np.max(np.abs(out[0][sample].cpu().numpy() - ref)) / max(1.0, np.max(np.abs(ref))))
    res = dict(
        metric="decode-attention requests/sec (one query token per request, one layer's KV cache per call)",
        value=n_req * layers / (ms * 1e-3), unit="requests/s", n_gpus=1, steps=steps, warmup=warmup,
        ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16", data="synthetic",
        config=dict(workload="decode attention, %d KV heads x %d query heads each x 128, %d requests, cache lengths U[%d, %d]" % (H, G, n_req, lo, hi),
                    calls_per_step=layers, kv_tokens=int(kv_len.sum()), accumulate="fp32",
                    l2="inputs larger than L2: a step streams %.2f GB of KV cache" % (kv_bytes / 1e9)),
        clocks=clocks, gpu_launches=3 * layers * steps,
        roofline=dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=achieved / peaks["hbm_gbs"],
                      traffic=NCU_ATTN_TRAFFIC_BYTES[long_ctx] * layers if G == 1 and not args.attn_requests else None,
                      traffic_from_build=NCU_TRAFFIC_BUILD if G == 1 and not args.attn_requests else None,
                      kernel="attn partial_kernel (chunked partial softmax)", peak_source=peaks["source"],
                      read_peak=read_gbs, frac_of_read_peak=None if read_gbs is None else achieved / read_gbs,
                      algorithmic_bytes_per_step=kv_bytes + other),
        cpu_baseline=dict(value=len(sample) / cpu_s, unit="requests/s", cores=1, kind="oracle",
                          sample="%d requests of one layer, numpy float64" % len(sample)),
        parity_max_rel_err=err, device_status=status)
    del q, K, V, out, ws
    torch.cuda.empty_cache()
    return res


def run_attention(args):
    print(json.dumps(attention_entry(args, long_ctx=args.attn_long, steps=args.steps)), flush=True)


# ----------------------------------------------------------------------------------
# starting the ranks of one node from this script
# ----------------------------------------------------------------------------------
def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_entry(rank: int, world: int, port: int, fn, fn_args):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    fn(*fn_args)


def spawn_local(world: int, fn, fn_args=()):
    """One process per rank on this node, each with the environment a launcher would give it (RANK,
    LOCAL_RANK, WORLD_SIZE, MASTER_ADDR, MASTER_PORT); returns when all have ended.  `fn` must be a
    module-level function."""
    import torch.multiprocessing as mp
    mp.spawn(_rank_entry, args=(world, _free_port(), fn, tuple(fn_args)), nprocs=world, join=True)


# ----------------------------------------------------------------------------------
# tensor-parallel adapter wave (paper Section VIII, Finding 5): row-parallel A, an all-reduce of the
# n_tok x rank intermediate, column-parallel B
# ----------------------------------------------------------------------------------
class KernelWave:
    """This rank's shard of every pool registered in the library; a step is bucket + one wave per pool:
    plora_shrink, all-reduce of m over the process group, plora_expand."""

    def __init__(self, wl, rank: int, world: int, local: int):
        import torch
        import torch.distributed as dist
        import paper_2608_05483_b200 as P
        from paper_2608_05483_b200.tp import TensorParallelDelta, shard_bounds
        self.torch, self.wl, self.rank, self.world = torch, wl, rank, world
        self.dev = f"cuda:{local}"
        torch.cuda.set_device(local)
        self.ctx = P.Context(wl.n_tok, wl.n_adapters, device=local)
        reduce = (lambda m: dist.all_reduce(m)) if world > 1 else (lambda m: None)
        self.tp = TensorParallelDelta(self.ctx, rank, world, reduce)
        self.ids = torch.from_numpy(wl.ids).to(self.dev)
        g = torch.Generator(device=self.dev)
        g.manual_seed(wl.seed)                 # the same draws on every rank: each keeps its columns
        self.x, self.y, self.bounds = {}, {}, {}
        self.pool_bytes = 0
        for pool in wl.pools:
            A, B = gen_pool_device(wl, pool, self.dev)
            slab = self.tp.register_pool(pool.layer, pool.proj, pool.d_in, pool.d_out, wl.ranks, wl.scales, A, B)
            self.pool_bytes += int(slab.numel())
            del A, B
            lo_i, hi_i = shard_bounds(pool.d_in, rank, world)
            lo_o, hi_o = shard_bounds(pool.d_out, rank, world)
            self.bounds[(pool.layer, pool.proj)] = (lo_i, hi_i, lo_o, hi_o)
            key = (pool.layer, pool.x_group)
            if key not in self.x:
                full = torch.randn((wl.n_tok, pool.d_in), generator=g, device=self.dev, dtype=torch.float32).to(torch.bfloat16)
                self.x[key] = (full, full[:, lo_i:hi_i].contiguous())
            full_y = torch.randn((wl.n_tok, pool.d_out), generator=g, device=self.dev, dtype=torch.float32)
            self.y[(pool.layer, pool.proj)] = full_y[:, lo_o:hi_o].contiguous()
        self.allreduce_bytes_per_wave = wl.n_tok * self.ctx.pool_max_rank(wl.pools[0].layer, wl.pools[0].proj) * 4
        torch.cuda.synchronize()

    def step(self):
        self.ctx.bucket(self.ids, self.wl.n_adapters)
        for p in self.wl.pools:
            self.tp.lora_delta(self.x[(p.layer, p.x_group)][1], self.ids, p.layer, p.proj, self.y[(p.layer, p.proj)])

    def timed(self, steps: int) -> float:
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            self.step()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    def launches(self) -> int:
        return self.ctx.launch_count()

    def check(self) -> float:
        """This rank's columns of y for the first pool against the oracle (full x and A, its columns of B)."""
        import oracle
        torch, wl = self.torch, self.wl
        pool = wl.pools[0]
        lo_i, hi_i, lo_o, hi_o = self.bounds[(pool.layer, pool.proj)]
        distinct = wl.distinct_adapters()
        A, B = gen_pool_device(wl, pool, self.dev)
        hA, hB = [None] * wl.n_adapters, [None] * wl.n_adapters
        for a in distinct:
            hA[int(a)] = bits_of(A[int(a)])
            hB[int(a)] = bits_of(B[int(a)][:, lo_o:hi_o])
        del A, B
        x_full = bits_of(self.x[(pool.layer, pool.x_group)][0])
        y_in = self.y[(pool.layer, pool.proj)].cpu().numpy().copy()
        want = oracle.lora_delta(x_full, wl.ids, wl.ranks, wl.scales, hA, hB, hi_o - lo_o, y_in)
        y = self.y[(pool.layer, pool.proj)].clone()
        self.ctx.bucket(self.ids, wl.n_adapters)
        self.tp.lora_delta(self.x[(pool.layer, pool.x_group)][1], self.ids, pool.layer, pool.proj, y)
        torch.cuda.synchronize()
        return float(np.max(np.abs(y.cpu().numpy() - want)) / np.max(np.abs(want - y_in)))

    def close(self):
        self.ctx.close()


def kernel_wave(wl, rank, world, local):
    return KernelWave(wl, rank, world, local)


def tp_job(args, make_wave=kernel_wave, result_path=None):
    """One rank of the tensor-parallel benchmark.  make_wave(wl, rank, world, local) builds the rank's wave
    (the library's kernels by default; the CPU test of the rank plumbing passes one that needs no GPU);
    rank 0 prints the JSON line and, if result_path is given, also writes it there."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    backend = args.tp_backend
    if world > 1:
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
        else:
            dist.init_process_group(backend)
    cfg = args.config or 2
    wl = make_workload(cfg, n_layers=args.layers or (1 if cfg == 1 else 4))
    wave = make_wave(wl, rank, world, local)
    red_dev = f"cuda:{local}" if backend == "nccl" else "cpu"
    err = max_over_ranks(wave.check(), red_dev)           # parity before anything is timed, worst rank
    warmup = max(3, args.warmup)
    for _ in range(warmup):
        wave.step()
    if world > 1:
        dist.barrier()
    l0 = wave.launches()
    ms = max_over_ranks(wave.timed(args.steps), red_dev)
    launches = wave.launches() - l0
    if world > 1:
        dist.barrier()
    if rank == 0:
        n_calls = len(wl.pools)
        out = dict(metric="LoRA-delta tokens/sec, tensor-parallel adapter wave (bucket + shrink, all-reduce of m, expand per pool)",
                   value=wl.n_tok / (ms * 1e-3), unit="tokens/s", n_gpus=world, steps=args.steps, warmup=warmup,
                   ms_per_step=ms, higher_is_better=True, scaling="strong", vs_baseline=None, dtype="bf16", data="synthetic",
                   config=dict(workload=f"config {cfg} ({wl.name})", n_tok=wl.n_tok, n_adapters=wl.n_adapters,
                               layers=len({p.layer for p in wl.pools}), calls_per_step=n_calls, parallelism=f"tp{world}",
                               collective=f"all-reduce of fp32 [n_tok, rank] per pool ({backend})"),
                   per_gpu_pool_bytes=wave.pool_bytes, allreduce_bytes_per_wave=wave.allreduce_bytes_per_wave,
                   allreduce_bytes_per_step=wave.allreduce_bytes_per_wave * n_calls, gpu_launches=int(launches),
                   parity_max_rel_err=err)
        line = json.dumps(out)
        print(line, flush=True)
        if result_path:
            Path(result_path).write_text(line)
    wave.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="lora", choices=["lora", "attention"],
                    help="lora: the LoRA-delta benchmark (the default, the headline); attention: decode attention")
    ap.add_argument("--attn-long", action="store_true", dest="attn_long", help="attention: 64 requests of 2048..4096 tokens")
    ap.add_argument("--attn-layers", type=int, default=4, dest="attn_layers")
    ap.add_argument("--attn-requests", type=int, default=0, dest="attn_requests")
    ap.add_argument("--attn-q-per-kv", type=int, default=1, choices=[1, 2, 4, 8], dest="attn_q_per_kv",
                    help="attention: query heads per KV head (1 = the Llama-2 7B / 13B shapes)")
    ap.add_argument("--gpus", type=int, default=1,
                    help="ranks of this node, one GPU each; started by this script unless a launcher's environment is there")
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None, choices=[1, 2, 3, 4, 5, 6],
                    help="one workload only (default: config 2 as the headline, then the others under per_config)")
    ap.add_argument("--layers", type=int, default=None)
    ap.add_argument("--graph", type=int, default=1)
    ap.add_argument("--cpu-pools", type=int, default=64, dest="cpu_pools")
    ap.add_argument("--cpu-seconds", type=float, default=20.0, dest="cpu_seconds",
                    help="target CPU time of the oracle sample (cpu_baseline leg)")
    ap.add_argument("--path", default="auto", choices=["auto", "fused", "unfused", "sgmv", "sgmv_split"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16"], help="16-bit type of x, A and B (fp16 = the paper's own)")
    ap.add_argument("--resident", type=int, default=1, choices=[0, 1],
                    help="1: tell the library that the step's inputs are resident before the step starts (plora_set_inputs_resident)")
    ap.add_argument("--no-group", action="store_true", dest="no_group",
                    help="one call per projection instead of grouping q/k/v and up/gate")
    ap.add_argument("--no-cpu", action="store_true", dest="no_cpu")
    ap.add_argument("--no-e2e", action="store_true", dest="no_e2e")
    ap.add_argument("--no-extras", action="store_true", dest="no_extras", help="headline only: no per_config entries")
    ap.add_argument("--no-read-peak", action="store_true", dest="no_read_peak",
                    help="skip the read-bandwidth probe (4 GiB of device memory): for profiler captures of a small case")
    ap.add_argument("--adapters", type=int, default=None,
                    help="adapters in every pool (default: the workload's 1000): a smaller pool for profiler captures, "
                         "the launch shape per adapter touched is unchanged")
    ap.add_argument("--tp", action="store_true",
                    help="the tensor-parallel adapter wave over --gpus ranks instead of replicas of the step")
    ap.add_argument("--tp-backend", default="nccl", choices=["nccl", "gloo"], dest="tp_backend")
    args = ap.parse_args()
    if args.op == "attention":
        run_attention(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        target = tp_job if args.tp else run_ours
        if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
            spawn_local(args.gpus, target, (args,))     # no launcher: this script starts the ranks
        else:
            target(args)


if __name__ == "__main__":
    main()
