#!/usr/bin/env python
"""Benchmark of the block-wise prefill hot path (append, attention, score, select, compact).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C5] [--mode graph|direct|batched]
  python bench.py --impl reference ...      # the CPU oracle as the reference arm

The default workload is C5 (long video), the largest single-GPU configuration and the one in which a launch
carries enough work for the roofline targets to be assessed.  At N = 1 the same JSON line carries, under
"workloads", the other bf16 configurations (C2, C3, C4 and the block-size study's T4), each measured the same way
with fewer steps (--no-extra skips them).

One "step" is one pass of the whole hot path over one synthetic request: every block of the
workload's prefix through every layer, starting from empty caches.  Prints ONE JSON line.

Modes (all run the same kernels through the C ABI):
  direct   one kvc_prefill_chunk call per (block, layer), issued from Python each step
  graph    the same calls captured once into a CUDA graph and replayed (no host work per step)
  batched  one kvc_prefill_chunk_layers call per block, the layer index in the launch grid
           (possible only because the synthetic q/k/v of all layers exist up front)
In the direct and graph modes a layer's score / select / compact is enqueued on the library's side stream
(KVC_FLAG_ASYNC_COMPRESS) and overlaps the next layer's attention, as it would in a decoder stack, where the
next layer waits for this layer's output and not for its compacted cache; the step ends after kvc_join, when
all of it has finished.  --sync-compress keeps everything in stream order.  Per-kernel durations are taken
in stream order, every kernel alone on the GPU.
With N > 1 every rank runs an independent replica of the request on its own GPU: the path has no
cross-GPU exchange, so there is no collective inside the timed region (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_16734_b200.workloads import CONFIGS, Workload  # noqa: E402

METRIC = "prefill tokens/s (attn+compress) per layer"
UNIT = "tokens/s/layer"
STEPS = ("append", "attention", "score", "compress")


# ------------------------------------------------------------------------------------------------
# peaks (roofline denominators)

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------------
# DRAM traffic of one steady-state launch (dram__bytes_read.sum + dram__bytes_write.sum of an ncu capture),
# kept as text under profiles/ together with a hash of the CUDA sources it was taken from; it is reported as
# null once the sources have changed.  File format: a line "sources <hash>", then "<workload> <kernel> <bytes>".

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.txt")


def kernel_sources_hash():
    """Hash of the CUDA sources with comments and white space removed (a reworded comment is not a new kernel)."""
    import glob
    import hashlib
    import re
    h = hashlib.sha256()
    for f in sorted(glob.glob(os.path.join(ROOT, "paper_2604_16734_b200", "csrc", "*"))):
        with open(f) as fh:
            text = fh.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update(re.sub(r"\s+", "", text).encode())
    return h.hexdigest()[:16]


def ncu_traffic(workload, kernel):
    try:
        with open(TRAFFIC_FILE) as f:
            rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None
    table = {(r[0], r[1]): int(r[2]) for r in rows if len(r) == 3}
    src = next((r[1] for r in rows if len(r) == 2 and r[0] == "sources"), None)
    if src != kernel_sources_hash():
        return None
    return table.get((workload, kernel))


# ------------------------------------------------------------------------------------------------
# algorithmic work of one launch (what the method itself has to move / compute)

def work_of_call(cfg, n, n_c, moves_per_head=None, fused_score=True, n_proxy=0):
    """Bytes and FLOPs per step kind for ONE layer of one kvc_prefill_chunk call (n includes the proxies)."""
    Hq, Hkv, d, sz, B = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.elem_bytes, cfg.budget
    tot = n_c + n - n_proxy
    w = n_proxy if n_proxy else min(cfg.obs_window, n)
    out = {}
    out["append"] = dict(bytes=2 * 2 * n * d * sz * Hkv + 4 * n * Hkv, flops=0)
    out["attention"] = dict(bytes=2 * (n_c + n) * d * sz * Hkv + 2 * n * d * sz * Hq + 4 * Hq * n,
                            flops=4 * Hq * d * (n * n_c + n * (n + 1) // 2))
    if tot > B:
        m = min(n, tot - B) * Hkv if moves_per_head is None else int(sum(moves_per_head))
        score = dict(bytes=Hkv * (tot - w) * d * sz + Hq * w * d * sz + 4 * Hq * w + 4 * Hkv * (tot - w),
                     flops=2 * Hq * w * d * (tot - w))
        select = 2 * 4 * Hkv * (tot - w) + 8 * m
        compact = m * (2 * 2 * d * sz + 8 + 8)
        if fused_score:          # one kernel scores, selects and compacts
            out["compress"] = dict(bytes=score["bytes"] + select + compact, flops=score["flops"])
        else:
            out["score"] = score
            out["compress"] = dict(bytes=select + compact, flops=0)
    return out


# ------------------------------------------------------------------------------------------------
# clocks

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.marks = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu=timestamp,{self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu_index)], stdout=self.file,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def mark(self):
        self.marks.append(time.time())

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.file.flush()
        rows = []
        try:
            with open(self.file.name) as f:
                for line in f:
                    parts = [x.strip() for x in line.split(",")]
                    if len(parts) >= 10:
                        rows.append(parts)
        finally:
            try:
                os.unlink(self.file.name)
            except OSError:
                pass
        return rows

    def summary(self, rows, t0, t1):
        import datetime
        sel = []
        for r in rows:
            try:
                ts = datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
            except ValueError:
                continue
            if t0 - 0.05 <= ts <= t1 + 0.05:
                sel.append(r)
        used = sel if sel else rows
        if not used:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        sm = [float(r[2]) for r in used]
        reasons = set()
        for r in used:
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[6:10]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=float(used[0][3]), reasons=sorted(reasons),
                    samples=len(sel), power_w_max=max(float(r[4]) for r in used))


# ------------------------------------------------------------------------------------------------
# the reference arm: the CPU oracle on a bounded sample

def oracle_sample_plan(cfg):
    """(layers, kv_heads, chunks) of the bounded sample the oracle runs per step."""
    sched = cfg.chunks()
    if cfg.name in ("C1", "C2"):
        return [0], None, sched, "layer 0, all kv-heads, whole prefix"
    if cfg.name == "C3":
        return [0], [0], sched, "layer 0, kv-head 0 of 4, whole prefix (scaled by 4)"
    # video: the per-block cost is flat once the cache is full; sample the first blocks past the budget
    n_fill = next(i for i, (p, n) in enumerate(sched) if p + n > cfg.budget) + 3
    return [0], [0], sched[:n_fill], f"layer 0, kv-head 0 of {cfg.n_kv_heads}, first {n_fill} blocks (scaled by {cfg.n_kv_heads})"


def run_oracle_sample(cfg, tensors_cpu, keep_out=None):
    """Times the oracle on the bounded sample.  With `keep_out` (a list) the outputs of the sampled blocks are appended
    to it as (pos0, n, query heads, out[n][heads][d]) for the caller to compare with what the GPU wrote."""
    from oracle.kvc_oracle import KVCOracle
    layers, heads, chunks, desc = oracle_sample_plan(cfg)
    orc = KVCOracle(1, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.budget, cfg.obs_window)
    q, k, v = tensors_cpu
    G = cfg.n_q_heads // cfg.n_kv_heads
    qh = list(range(cfg.n_q_heads)) if heads is None else [g * G + j for g in heads for j in range(G)]
    t0 = time.perf_counter()
    tokens = 0
    for pos0, n in chunks:
        res = orc.prefill_chunk(0, q[pos0:pos0 + n], k[pos0:pos0 + n], v[pos0:pos0 + n], pos0, kv_heads=heads)
        if keep_out is not None:
            keep_out.append((pos0, n, qh, res.out[:, qh, :]))
        tokens += n
    dt = time.perf_counter() - t0
    frac_heads = 1.0 if heads is None else len(heads) / cfg.n_kv_heads
    return tokens * len(layers) * frac_heads / dt, dt, desc


def check_outputs(O_layer, kept, bf16):
    """Compares the attention outputs the GPU left for one layer with the oracle's on the sampled blocks: plain
    max-abs error against the output tolerance (1e-4 fp32, 2e-2 bf16), and for bf16 how many elements beyond it are
    within one bf16 unit in the last place of the oracle value rounded to bf16 (the only escape the parity tests
    allow).  Both sides run free here: a near-tie at an eviction that the two resolve differently shows up as an
    error in the blocks after it (the parity tests adopt the oracle's set instead)."""
    tol = 2e-2 if bf16 else 1e-4
    worst, ref_max, n_cmp, n_over, n_ulp = 0.0, 0.0, 0, 0, 0
    for pos0, n, qh, ref in kept:
        got = O_layer[pos0:pos0 + n][:, qh, :].double().cpu().numpy()
        err = np.abs(got - ref)
        worst = max(worst, float(err.max())); ref_max = max(ref_max, float(np.abs(ref).max())); n_cmp += err.size
        over = err > tol
        if over.any():
            n_over += int(over.sum())
            if bf16:
                r16 = torch.from_numpy(ref[over]).to(torch.bfloat16)
                ulp = (r16.abs().double().clamp_min(2.0 ** -126).log2().floor() - 7).exp2().numpy()
                n_ulp += int((np.abs(got[over] - r16.double().numpy()) <= ulp).sum())
    return dict(max_abs_err=worst, tolerance=tol, max_abs_ref=ref_max, elements=n_cmp, beyond_tolerance=n_over,
                of_those_within_one_bf16_ulp=n_ulp, ok=bool(n_over == n_ulp))


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def config_dict(cfg, L, args, world, extra=None):
    """The `config` object of the JSON line: the same keys for both arms."""
    d = {"workload": cfg.name, "layers": L, "q_heads": cfg.n_q_heads, "kv_heads": cfg.n_kv_heads,
         "head_dim": cfg.head_dim, "tokens": cfg.n_tokens, "block": cfg.chunk, "budget": cfg.budget,
         "obs_window": cfg.obs_window, "policy": args.policy, "schedule": "hybrid" if args.hybrid else "block-wise",
         "proxy_tokens": args.proxy, "mode": args.mode, "parallelism": f"replicas x{world}"}
    if extra:
        d.update(extra)
    return d


def reference_arm(args, cfg, rank):
    if rank != 0:
        return
    wl = Workload(cfg, device="cpu")
    q, k, v = wl.layer(0)
    tens = (q.double().numpy(), k.double().numpy(), v.double().numpy())
    for _ in range(args.warmup):
        run_oracle_sample(cfg, tens)
    vals, times = [], []
    desc = ""
    for _ in range(args.steps):
        val, dt, desc = run_oracle_sample(cfg, tens)
        vals.append(val); times.append(dt)
    value = sum(vals) / len(vals)
    L = args.layers if args.layers else cfg.n_layers
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(cfg, L, args, int(os.environ.get("WORLD_SIZE", "1")),
                                  {"compress": "n/a (CPU oracle)", "l2": "n/a (CPU oracle)", "sample": desc}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# our arm

class Runner:
    def __init__(self, cfg, device_index, n_layers=None, flags=0, policy=0, hybrid=False, proxy=0):
        from paper_2604_16734_b200.binding import Kvc
        self.cfg = cfg
        self.flags = flags
        self.policy = policy
        self.L = cfg.n_layers if n_layers is None else n_layers
        self.dev = torch.device("cuda", device_index)
        wl = Workload(cfg, device=self.dev)
        N = cfg.n_tokens
        self.Q = torch.empty(self.L, N, cfg.n_q_heads, cfg.head_dim, dtype=cfg.torch_dtype, device=self.dev)
        self.K = torch.empty(self.L, N, cfg.n_kv_heads, cfg.head_dim, dtype=cfg.torch_dtype, device=self.dev)
        self.V = torch.empty_like(self.K)
        for l in range(self.L):
            q, k, v = wl.layer(l)
            self.Q[l], self.K[l], self.V[l] = q, k, v
        del wl
        self.sched = cfg.chunks_hybrid() if hybrid else cfg.chunks()
        # calls: (row offset in the buffers, rows of the call, proxy rows among them, position of the first token)
        self.calls = [(p, n, 0, p) for p, n in self.sched]
        self.proxy = proxy
        if proxy:
            # proxy query tokens (Sec. 3.2): the first `proxy` text tokens follow every vision block in the input
            # buffers, so that a call's rows stay contiguous; the text prompt is an ordinary block at the end
            nv = cfg.n_vision
            assert 0 < proxy <= cfg.n_text
            idx, calls, off = [], [], 0
            for p, n in self.sched:
                t = proxy if p < nv else 0
                idx.append(torch.arange(p, p + n, device=self.dev))
                if t:
                    idx.append(torch.arange(nv, nv + t, device=self.dev))
                calls.append((off, n + t, t, p))
                off += n + t
            idx = torch.cat(idx)
            self.Q, self.K, self.V = (x[:, idx].contiguous() for x in (self.Q, self.K, self.V))
            self.calls = calls
        self.O = torch.empty_like(self.Q)
        self.kvc = Kvc(self.L, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.budget, cfg.chunk + proxy,
                       cfg.obs_window, device=device_index, flags=flags, policy=policy)
        # per-kernel timing wants every kernel alone on the GPU: a second context that keeps compress in stream order
        self.kvc_in_order = self.kvc if not flags & 16 else Kvc(
            self.L, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.budget, cfg.chunk + proxy,
            cfg.obs_window, device=device_index, flags=flags & ~16, policy=policy)
        # raw pointers of every (block, layer) slice, so the per-call host work is one ctypes call
        self.ptrs = {}
        for ci, (o, n, t, p) in enumerate(self.calls):
            for l in range(self.L):
                self.ptrs[ci, l] = (self.Q[l, o:o + n].data_ptr(), self.K[l, o:o + n].data_ptr(),
                                    self.V[l, o:o + n].data_ptr(), self.O[l, o:o + n].data_ptr())
        self.graph = None

    def step_direct(self):
        kv, lib, h = self.kvc, self.kvc._lib, self.kvc._h
        st = kv._stream()
        kv.reset()
        ws = kv.workspace.data_ptr()
        cache0, blob = kv.cache.data_ptr(), kv.blob_bytes
        for ci, (_, n, t, p) in enumerate(self.calls):
            for l in range(self.L):
                q, k, v, o = self.ptrs[ci, l]
                if t:
                    rc = lib.kvc_prefill_chunk_proxy(h, l, q, k, v, n, t, p, cache0 + l * blob, ws, o, st)
                else:
                    rc = lib.kvc_prefill_chunk(h, l, q, k, v, n, p, cache0 + l * blob, ws, o, st)
                if rc:
                    kv._check(rc)
        if self.flags & 16:              # compress kernels on the side stream: the step ends when they have
            kv.join()

    def step_batched(self):
        kv = self.kvc
        kv.reset()
        for p, n in self.sched:
            kv.prefill_chunk_layers(0, self.Q[:, p:p + n], self.K[:, p:p + n], self.V[:, p:p + n], p, self.O[:, p:p + n])

    def capture(self):
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.step_direct()

    def step_graph(self):
        self.graph.replay()

    def step_host(self, host):
        """End-to-end: q/k/v from pinned host memory, out back to pinned host memory, every call."""
        kv = self.kvc
        kv.reset()
        qh, kh, vh, oh = host
        for p, n in self.sched:
            for l in range(self.L):
                kv.prefill_chunk_host(l, qh[l, p:p + n], kh[l, p:p + n], vh[l, p:p + n], p, oh[l, p:p + n])
        kv.host_flush()                                       # the step ends when the last result is on the host


def max_over_ranks(seconds: float, dist, device) -> float:
    """The job is as slow as its slowest rank: MAX-reduce a duration over the process group (if any)."""
    if dist is None:
        return seconds
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_layer: int, layers: int, steps: int, world: int, seconds: float) -> float:
    """Metric of the whole job: every rank runs a replica of the request (weak scaling), so the tokens x layers
    all ranks processed in `steps` steps, divided by the time of the slowest rank."""
    return world * tokens_per_layer * layers * steps / seconds


def time_steps(fn, steps, barrier):
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    barrier()
    return e0.elapsed_time(e1) / 1e3, t0, t1


def stamps_as_timed(r: Runner):
    """Device time stamps of one step in the configuration the benchmark times (compress kernels on the library's
    side streams when the context has them; calls issued directly, not from the graph): per kernel its launches, mean
    duration, total and share.  On a side stream a compress kernel gets fewer CTAs per kv-head than in stream order
    and runs longer, beside the next layer's attention -- this is the table the ncu launch list of the same command
    compares with."""
    kv = r.kvc
    r.step_direct()
    torch.cuda.synchronize()
    before = kv.launch_count()
    r.step_direct()
    torch.cuda.synchronize()
    per_step = kv.launch_count() - before
    kv.profile_device(per_step + 16)
    r.step_direct()
    ms, cnt, span_ms = kv.profile_device_read()
    kv.profile_device(0)
    tot = sum(ms.values())
    return {s: dict(launches_per_step=cnt[s], us_per_launch=1e3 * ms[s] / cnt[s], ms_total_per_step=ms[s],
                    share=ms[s] / tot) for s in ms if cnt[s]} | {"span_ms": span_ms}


def profile_pass(r: Runner, steps: int, batched: bool = False, events: bool = False):
    """Per-kernel durations and exact algorithmic work: one call per (block, layer), in stream order, or with
    `batched` one call per block with the layer index in the launch grid.  The durations are device-side time
    stamps taken inside the kernels (global timer; per launch from the earliest begin of work, past the wait for
    the preceding kernel, to the latest end over its CTAs): no event pair sits between consecutive launches, so
    they overlap as they do in the timed step, and the sum of the durations fits inside the step."""
    saved = (r.kvc, r.flags)
    r.kvc, r.flags = r.kvc_in_order, r.flags & ~16
    kv, cfg = r.kvc, r.cfg
    work = {s: dict(bytes=0, flops=0) for s in STEPS}
    # exact move counts need one pass with a readback after every call
    kv.reset()
    n_c = 0
    for ci, (_, n, t, p) in enumerate(r.calls):
        for l in range(r.L):
            q, k, v, o = r.ptrs[ci, l]
            if t:
                kv._check(kv._lib.kvc_prefill_chunk_proxy(kv._h, l, q, k, v, n, t, p, kv.cache[l].data_ptr(),
                                                          kv.workspace.data_ptr(), o, kv._stream()))
            else:
                kv._check(kv._lib.kvc_prefill_chunk(kv._h, l, q, k, v, n, p, kv.cache[l].data_ptr(), kv.workspace.data_ptr(),
                                                    o, kv._stream()))
            moves = kv.move_counts(0).tolist() if n_c + n - t > cfg.budget else None
            w_call = t if t else min(cfg.obs_window, n)
            fused = r.policy == 1 or (cfg.dtype == "bf16" and not (r.flags & 1) and w_call * cfg.group <= 128)
            for s, wv in work_of_call(cfg, n, n_c, moves, fused, t).items():
                work[s]["bytes"] += wv["bytes"]; work[s]["flops"] += wv["flops"]
        n_c = min(n_c + n - t, cfg.budget)
    torch.cuda.synchronize()
    per_step = kv.launch_count()
    (r.step_batched if batched else r.step_direct)()
    torch.cuda.synchronize()
    per_step = kv.launch_count() - per_step
    kv.profile_device(per_step * steps + 16)
    for _ in range(steps):
        (r.step_batched if batched else r.step_direct)()
    ms, cnt, span_ms = kv.profile_device_read()
    kv.profile_device(0)
    # the same launches bracketed by CUDA events on the launching stream (a pair per launch: each kernel alone on the
    # GPU, launch latency and the events themselves included)
    ev_ms = ev_cnt = None
    if events:
        kv.profile_enable(True)
        for _ in range(min(steps, 3)):
            (r.step_batched if batched else r.step_direct)()
        torch.cuda.synchronize()
        ev_ms, ev_cnt = kv.profile_read()
        kv.profile_enable(False)
    r.kvc, r.flags = saved
    per = {}
    for s in STEPS:
        if cnt[s]:
            per[s] = dict(ms_total_per_step=ms[s] / steps, launches_per_step=cnt[s] // steps,
                          us_per_launch=1e3 * ms[s] / cnt[s], bytes_per_step=work[s]["bytes"],
                          flops_per_step=work[s]["flops"])
            if ev_cnt and ev_cnt[s]:
                per[s]["us_per_launch_cuda_events"] = 1e3 * ev_ms[s] / ev_cnt[s]
    return per


def rates(per, peaks):
    for d in per.values():
        sec = d["ms_total_per_step"] / 1e3
        d["gbs"] = d["bytes_per_step"] / sec / 1e9
        d["tflops"] = d["flops_per_step"] / sec / 1e12
        d["hbm_frac"] = d["gbs"] / peaks["hbm_gbs"]
        d["tensor_frac_sustained"] = d["tflops"] / peaks["tflops_sustained"]
        d["tensor_frac_burst"] = d["tflops"] / peaks["tflops_burst"]
    return per


def step_roofline(cfg, per, L, ms_per_step, peaks):
    """The path's roofline for one step (all blocks x L layers), from the exact algorithmic work of the step: the
    slower of the attention at the measured bf16 peak (its own HBM time where that is longer, or its HBM time alone
    for fp32, which does not use the tensor cores) and the score / select / compact bytes at the measured HBM
    bandwidth; also the stricter sum of the two, since the steps of one layer run back to back."""
    att = per.get("attention")
    if not att:
        return None
    hbm = peaks["hbm_gbs"] * 1e9
    t_att_hbm = (att["bytes_per_step"] + per.get("append", {}).get("bytes_per_step", 0)) / hbm
    t_att_tc = att["flops_per_step"] / (peaks["tflops_sustained"] * 1e12) if cfg.dtype == "bf16" else 0.0
    t_att = max(t_att_hbm, t_att_tc)
    t_cmp = sum(per[s]["bytes_per_step"] for s in ("score", "compress") if s in per) / hbm
    bound, bound_sum = max(t_att, t_cmp), t_att + t_cmp
    meas = ms_per_step / 1e3
    return dict(bound_ms=1e3 * bound, bound_sum_ms=1e3 * bound_sum, measured_ms=ms_per_step, frac=bound / meas,
                frac_of_sum_bound=bound_sum / meas,
                attention_bound="tensor" if t_att_tc >= t_att_hbm else "hbm", attention_ms_at_peak=1e3 * t_att,
                compress_ms_at_hbm=1e3 * t_cmp,
                tokens_per_s_per_layer_at_bound=cfg.n_tokens * L / bound,
                peak_source=peaks["source"] + " (sustained bf16, copy bandwidth)")


def measure(cfg, args, L, local_rank, rank, world, dist, barrier, peaks, steps, primary):
    """Times one workload: the step as configured (`value`), the same step with every kernel in stream order, the
    kernels one by one, and (primary workload only) the end-to-end path from host buffers and the CPU oracle."""
    flags = args.flags
    side_stream = (args.mode != "batched" and not args.sync_compress and cfg.dtype == "bf16" and not flags & 1)
    if side_stream:
        flags |= 16
    r = Runner(cfg, local_rank, L, flags, 1 if args.policy == "keydiff" else 0, args.hybrid, args.proxy)
    kv = r.kvc
    sampler = ClockSampler(local_rank)
    sampler.start()

    step = {"direct": r.step_direct, "batched": r.step_batched, "graph": r.step_graph}[args.mode]
    (r.step_batched if args.mode == "batched" else r.step_direct)()   # sets function attributes, resolves the driver entry point
    torch.cuda.synchronize()
    if args.mode == "graph":
        r.capture()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert kv.status() == 0, kv.last_error()
    launches_before = kv.launch_count()
    if args.mode == "graph":              # a replay launches what one captured step launched
        r.step_direct(); torch.cuda.synchronize()
        launches_per_step = kv.launch_count() - launches_before
    secs, t0, t1 = time_steps(step, steps, barrier)
    if args.mode != "graph":
        launches_per_step = (kv.launch_count() - launches_before) // steps
    assert kv.status() == 0, kv.last_error()
    secs = max_over_ranks(secs, dist, "cuda")
    rows = sampler.stop()
    clocks = sampler.summary(rows, t0, t1)
    value = whole_job_value(cfg.n_tokens, L, steps, world, secs)
    ms_per_step = 1e3 * secs / steps
    out = dict(value=value, ms_per_step=ms_per_step, steps=steps, launches_per_step=launches_per_step, clocks=clocks)

    # ---- the same step with every kernel in stream order (no side streams): the serial chain of the launches
    in_order_ms = None
    if rank == 0 and not args.no_profile:
        if side_stream and args.mode in ("graph", "direct"):
            saved = (r.kvc, r.flags, r.graph)
            r.kvc, r.flags = r.kvc_in_order, r.flags & ~16
            r.step_direct(); torch.cuda.synchronize()
            if args.mode == "graph":
                r.capture()
            fn = r.step_graph if args.mode == "graph" else r.step_direct
            for _ in range(2):
                fn()
            n_io = max(3, min(steps, 10))
            io_secs, _, _ = time_steps(fn, n_io, lambda: None)
            in_order_ms = 1e3 * io_secs / n_io
            r.kvc, r.flags, r.graph = saved
        else:
            in_order_ms = ms_per_step
        out["ms_per_step_in_order"] = in_order_ms

    # ---- per-kernel durations and rooflines (rank 0, outside the timed region)
    per, per_b, roof = {}, {}, None
    if rank == 0 and not args.no_profile:
        per = rates(profile_pass(r, max(3, min(steps, 10)) if primary else 3, events=True), peaks)
        ridge = peaks["tflops_sustained"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
        dom = max(per, key=lambda s: per[s]["ms_total_per_step"])
        d = per[dom]
        ai = d["flops_per_step"] / max(d["bytes_per_step"], 1)
        # `achieved` rests on CUDA events around every launch of the kernel (the slower, self-contained figure: launch
        # latency and the events are inside it); the device-stamped duration, which is what the launch occupies in the
        # in-order step, is given beside it
        ev_sec = d.get("us_per_launch_cuda_events", d["us_per_launch"]) * 1e-6 * d["launches_per_step"]
        ev_tflops, ev_gbs = d["flops_per_step"] / ev_sec / 1e12, d["bytes_per_step"] / ev_sec / 1e9
        if cfg.dtype == "bf16" and dom == "attention" and ai > ridge:
            # the kernel is timed inside a long step: the sustained peak is its denominator; the burst figure beside it
            roof = dict(kernel=dom, bound="tensor", achieved=ev_tflops, peak=peaks["tflops_sustained"], unit="TFLOP/s",
                        frac=ev_tflops / peaks["tflops_sustained"], traffic=None,
                        peak_source=peaks["source"] + " (sustained bf16)", peak_burst=peaks["tflops_burst"],
                        frac_of_burst_peak=ev_tflops / peaks["tflops_burst"],
                        achieved_device_stamps=d["tflops"], frac_device_stamps=d["tflops"] / peaks["tflops_sustained"],
                        frac_of_burst_peak_device_stamps=d["tflops"] / peaks["tflops_burst"])
        else:
            roof = dict(kernel=dom, bound="hbm", achieved=ev_gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=ev_gbs / peaks["hbm_gbs"], traffic=None, peak_source=peaks["source"],
                        achieved_device_stamps=d["gbs"], frac_device_stamps=d["gbs"] / peaks["hbm_gbs"])
        roof["traffic"] = ncu_traffic(cfg.name, dom) if L == cfg.n_layers else None
        roof["algorithmic_bytes_per_launch"] = d["bytes_per_step"] / max(d["launches_per_step"], 1)
        roof["algorithmic_flops_per_launch"] = d["flops_per_step"] / max(d["launches_per_step"], 1)
        roof["us_per_launch"] = d.get("us_per_launch_cuda_events", d["us_per_launch"])
        roof["us_per_launch_device_stamps"] = d["us_per_launch"]
        roof["arithmetic_intensity"] = ai
        roof["timing"] = ("achieved / frac: CUDA events around every launch on the launching stream, kernels in stream order; "
                          "*_device_stamps: time stamps inside the kernel (global timer, earliest begin of work, past the wait "
                          "for the preceding kernel, to the latest end over the CTAs of a launch)")
        # the kernels' durations against the step they have to fit into
        kernel_ms_sum = sum(x["ms_total_per_step"] for x in per.values())
        out["kernel_ms_sum"] = kernel_ms_sum
        out["overlap"] = dict(
            ms_per_step_in_order=in_order_ms, ms_per_step=ms_per_step,
            hidden_by_side_streams_ms=(in_order_ms - ms_per_step) if in_order_ms is not None else None,
            kernel_ms_sum_over_in_order=kernel_ms_sum / in_order_ms if in_order_ms else None,
            note="kernel_ms_sum adds the device-stamped durations of all launches of an in-order step; what the in-order "
                 "step holds beyond it is the time between launches (launch latency, cache resets)")
        out["roofline_step"] = step_roofline(cfg, per, L, ms_per_step, peaks)
        if in_order_ms is not None and out["roofline_step"]:
            out["roofline_step"]["frac_in_order"] = out["roofline_step"]["bound_ms"] / in_order_ms
        # ---- the same kernels with all layers in one launch (possible only with synthetic inputs): what the
        #      bandwidth-bound steps reach when a launch carries enough bytes to fill the GPU
        if L > 1 and not args.proxy:
            per_b = rates(profile_pass(r, 3, batched=True), peaks)
    out["kernels"], out["kernels_layer_batched"], out["roofline"] = per, per_b, roof
    if rank == 0 and not args.no_profile and args.mode != "batched" and (flags & 16):
        out["kernels_as_timed"] = stamps_as_timed(r)

    # ---- end to end through the host-buffer entry point
    if primary and not args.no_e2e and not args.proxy:          # (the host-buffer entry point has no proxy variant)
        host = tuple(t.cpu().pin_memory() for t in (r.Q, r.K, r.V)) + (torch.empty(r.O.shape, dtype=r.O.dtype).pin_memory(),)
        for _ in range(2):
            r.step_host(host)
        torch.cuda.synchronize()
        e_steps = max(1, min(steps, 5))
        esecs, _, _ = time_steps(lambda: r.step_host(host), e_steps, barrier)
        esecs = max_over_ranks(esecs, dist, "cuda")
        h2d = sum(t.numel() * t.element_size() for t in host[:3])
        d2h = host[3].numel() * host[3].element_size()
        out["e2e"] = dict(value=world * cfg.n_tokens * L * e_steps / esecs, unit=UNIT, h2d_bytes_per_step=h2d,
                          d2h_bytes_per_step=d2h, steps=e_steps, ms_per_step=1e3 * esecs / e_steps)
        del host

    # ---- CPU baseline: the oracle on a bounded sample of the same workload (rank 0, N = 1)
    if primary and rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the same bounded sample on successive layers until about 10 s of CPU work have been spent
        tot_dt, vals, desc, nl_done = 0.0, [], "", 0
        kept = []
        while nl_done < L and tot_dt < 10.0:
            tens = tuple(t[nl_done].double().cpu().numpy() for t in (r.Q, r.K, r.V))
            val, dt, desc = run_oracle_sample(cfg, tens, kept if nl_done == 0 else None)
            vals.append(val); tot_dt += dt; nl_done += 1
        out["cpu_baseline"] = dict(value=len(vals) / sum(1.0 / x for x in vals), unit=UNIT, cores=cpu_threads(), kind="oracle",
                                   sample=desc.replace("layer 0", f"layers 0..{nl_done - 1}"), seconds=tot_dt)
        # the outputs of the measured configuration (whatever pass wrote them last: all passes give the same bits),
        # layer 0, against the oracle's on the same sample
        if not args.proxy and not args.hybrid and args.policy == "attn":
            out["output_check"] = dict(check_outputs(r.O[0], kept, cfg.elem_bytes == 2), sample=desc)

    logical, physical, full = kv.kv_bytes(cfg.n_tokens)
    out["kv_bytes"] = {"logical_budget": logical, "physical_allocated": physical, "uncompressed": full,
                       "blobs_incl_positions": kv.blob_bytes * L}
    out["config"] = config_dict(cfg, L, args, world, {
        "compress": "side stream, beside the next layer's attention" if flags & 16 else "in stream order",
        "l2": "inputs exceed L2" if (r.Q.numel() + 2 * r.K.numel()) * cfg.elem_bytes > 126e6 else "inputs fit L2"})
    r.kvc.close()
    if r.kvc_in_order is not r.kvc:
        r.kvc_in_order.close()
    del r
    torch.cuda.empty_cache()
    return out


EXTRA_WORKLOADS = ("C2", "C3", "C4", "T4")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C5", choices=sorted(CONFIGS))
    ap.add_argument("--mode", default="graph", choices=["graph", "direct", "batched"])
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (0 = all; not a headline run)")
    ap.add_argument("--block", type=int, default=0, help="override the workload's block size b (block-size study, Sec. 5 / Table 4)")
    ap.add_argument("--budget", type=int, default=0, help="override the workload's budget M")
    ap.add_argument("--proxy", type=int, default=0,
                    help="proxy query tokens (Sec. 3.2): the first PROXY text tokens ride along with every vision block as "
                         "observers and are never cached (graph / direct modes only)")
    ap.add_argument("--hybrid", action="store_true",
                    help="hybrid schedule (Sec. 5, Budgeting): the first B tokens in one pass, block-wise after that")
    ap.add_argument("--policy", default="attn", choices=["attn", "keydiff"],
                    help="eviction score: query-aware attention score (Eq. 4) or query-agnostic key similarity (Sec. 3.2)")
    ap.add_argument("--flags", type=int, default=0, help="KVC_FLAG_* bits passed to kvc_create (kernel selection, diagnostics)")
    ap.add_argument("--sync-compress", action="store_true",
                    help="keep a layer's score / select / compact in stream order behind its attention instead of "
                         "on the library's side stream (KVC_FLAG_ASYNC_COMPRESS, the default of the graph / direct modes)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-profile", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the other workloads reported under \"workloads\"")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = CONFIGS[args.workload]
    if args.block or args.budget:
        cfg = cfg.scaled(chunk=args.block or cfg.chunk, budget=args.budget or cfg.budget)
    if args.impl == "reference":
        reference_arm(args, cfg, rank)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    args.warmup = max(args.warmup, 3)
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if dist is not None:
            dist.barrier()

    peaks = load_peaks()
    L = args.layers if args.layers else cfg.n_layers
    if args.proxy and (args.mode == "batched"):
        raise SystemExit("--proxy runs in the graph and direct modes only")
    m = measure(cfg, args, L, local_rank, rank, world, dist, barrier, peaks, args.steps, primary=True)

    # ---- the other bf16 configurations, measured the same way (N = 1, default settings only)
    extra = {}
    plain = not (args.block or args.budget or args.proxy or args.hybrid or args.layers or args.flags or args.no_profile)
    if rank == 0 and world == 1 and not args.no_extra and plain and args.policy == "attn" and args.workload == "C5":
        for name in EXTRA_WORKLOADS:
            c2 = CONFIGS[name]
            x = measure(c2, args, c2.n_layers, local_rank, rank, world, None, lambda: None, peaks,
                        max(3, min(args.steps, 10)), primary=False)
            extra[name] = {k: x[k] for k in ("value", "ms_per_step", "ms_per_step_in_order", "steps", "launches_per_step",
                                             "kernel_ms_sum", "kernels", "kernels_layer_batched", "kernels_as_timed", "roofline", "roofline_step",
                                             "overlap", "kv_bytes", "clocks", "config") if k in x}
            extra[name]["unit"] = UNIT

    if rank == 0:
        line = {"metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic", "config": m["config"],
                "clocks": m["clocks"], "gpu_launches": m["launches_per_step"] * args.steps,
                "launches_per_step": m["launches_per_step"], "kv_bytes": m["kv_bytes"], "kernels": m["kernels"],
                "kernels_layer_batched": m["kernels_layer_batched"]}
        if "kernels_as_timed" in m:
            line["kernels_as_timed"] = m["kernels_as_timed"]
        for k in ("ms_per_step_in_order", "kernel_ms_sum", "overlap", "roofline_step", "e2e", "cpu_baseline", "output_check"):
            if k in m:
                line[k] = m[k]
        if m.get("roofline"):
            line["roofline"] = m["roofline"]
        if extra:
            line["workloads"] = extra
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
