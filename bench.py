#!/usr/bin/env python
"""Benchmark of the chunked instruction-aware eviction hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Headline workload: the long-document stress configuration (131072 tokens = 32 chunks of 4096; 32/8 heads,
head_dim 128, budget 4096, 256 instruction queries, bf16, individual caches, every chunk query scores the
language-modelling cache), the largest of the five named configurations that one GPU holds.  One step = R
passes of the whole document through a1-a4, chunk by chunk, replayed from a CUDA graph (R is chosen so that
the timed region lasts about two seconds, and is printed in `config`).

Prints ONE JSON line: document tokens/s (device-timed, inputs resident in HBM), the same metric end to end
through the host-buffer ABI call, the roofline of the attention kernel, the fp64 oracle timed on the host
cores, and a `configs` array with the same figures for all five named configurations.
With N > 1 every rank runs its own document: weak scaling, no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2406_12018_b200 import workloads as wl  # noqa: E402

WORKLOAD = "long_doc_stress"
# dram__bytes_read.sum + dram__bytes_write.sum of one steady-state launch of the attention kernel on the headline
# workload, from the ncu summary under profiles/; None whenever that kernel has changed since the capture.
ATTN_DRAM_TRAFFIC_BYTES = 102.4e6
ATTENTION_BESIDE = None          # --attention-beside: passed to every context (None = the library's default)
BATCH_LANES = 0                  # --lanes: passed to the contexts of batch workloads (0 = the library's choice)
METRIC = "document tokens/s through chunked eviction per layer"
UNIT = "tokens/s"
TARGET_TIMED_SECONDS = 2.2
ALL_WORKLOADS = {**wl.CONFIGS, **wl.PAPER_SHAPES, **wl.VARIANTS}


# --------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "hbm_gbs": d["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        # nvidia-smi numbers the GPUs of the machine, CUDA those that are visible to the process: ask by UUID
        try:
            self.idx = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
        except Exception:
            self.idx = device_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.idx)], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def wait_first_sample(self, timeout_s: float = 10.0):
        """nvidia-smi needs a moment to start: return once it has printed its first line."""
        t_end = time.time() + timeout_s
        while self.proc is not None and not self.lines and time.time() < t_end:
            time.sleep(0.05)

    def stop(self, t_begin: float = 0.0, t_end: float = float("inf")):
        """Summary of the samples taken in [t_begin, t_end] (host clock), the timed region."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for stamp, ln in self.lines:
            if not (t_begin <= stamp <= t_end):
                continue
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            try:
                pw.append(float(parts[3]))
            except ValueError:
                pass
            for nm, v in zip(names, parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "sm_mhz_min": min(sm) if sm else None, "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def chunk_bounds(n_tokens: int, chunk_s: int):
    return [(s, min(n_tokens, s + chunk_s)) for s in range(0, n_tokens, chunk_s)]


def step_sizes(w: wl.Workload, n_tokens: int):
    """(L, m) of every chunk step of one document: chunk rows and rows retained before the step."""
    seen, out = 0, []
    for a, b in chunk_bounds(n_tokens, w.chunk_s):
        out.append((b - a, min(w.budget_k, seen)))
        seen += b - a
    return out


def algorithmic_work(w: wl.Workload, sizes):
    """Algorithmic flops / bytes of one pass over chunk steps `sizes` = [(L, m)] (per layer, per sequence).

    a1: 4 D H_q (L m + L (L + 1) / 2) flops.   a2-I: 2 D H_q n_I n flops (one Q.K^T).
    a3: 4 n read + 4 kept written per (cache, KV head).
    a4: kept rows x D x elt x (K, V), read and written, + 8 bytes of positions per row, per (cache, KV head)."""
    elt = 2 if w.dtype == "bf16" else 4
    n_caches = 2 if w.mode == "individual" else 1
    a1 = a2 = a3 = a4 = 0.0
    for L, m in sizes:
        n, kept = m + L, min(w.budget_k, m + L)
        a1 += 4.0 * w.head_dim * w.q_heads * (L * m + L * (L + 1) / 2.0)
        if w.mode != "standard":
            a2 += 2.0 * w.head_dim * w.q_heads * w.n_instr * n
        a3 += n_caches * w.kv_heads * (4.0 * n + 4.0 * kept)
        a4 += n_caches * w.kv_heads * (2.0 * 2 * kept * w.head_dim * elt + 8.0 * kept)
    return {"a1_flops": a1, "a2i_flops": a2, "a3_bytes": a3, "a4_bytes": a4}


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


# --------------------------------------------------------------------------- oracle arm
def oracle_sample(w: wl.Workload):
    """The bounded sample the oracle is timed on: one chunk of `rows` tokens against a full cache."""
    rows = min(w.chunk_s, 512)
    return rows, (f"one chunk of {rows} tokens per step against a full cache of {w.budget_k} retained states"
                  f" ({w.mode} caches, {w.n_instr} instruction queries); a full chunk of this workload has {w.chunk_s} tokens")


def run_reference(args, rank):
    """The fp64 oracle, as it stands, on the host cores: rank 0 only, a bounded sample of the workload per step."""
    if rank != 0:
        return
    import oracle
    from threadpoolctl import threadpool_limits
    w = ALL_WORKLOADS[args.workload]
    threads = host_cores()
    rows, sample = oracle_sample(w)
    n_steps = args.steps + args.warmup
    doc = wl.make_document(w, n_tokens=w.budget_k + rows * n_steps)
    Q, K, V, Qi = (wl.to_f64(t) for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
    orc = oracle.CitrusOracle(w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.mode,
                              lm_window=(w.lm_window or None), layerwise=w.layerwise)
    # a full cache to start from: the document's first budget_k states (a valid retained set: full, ascending positions)
    k = w.budget_k
    for cid in range(len(orc.caches)):
        orc.caches[cid] = oracle.CacheState(np.ascontiguousarray(K[:k].transpose(1, 0, 2)),
                                            np.ascontiguousarray(V[:k].transpose(1, 0, 2)),
                                            np.broadcast_to(np.arange(k, dtype=np.int64), (w.kv_heads, k)).copy())
    orc.tokens_seen = k
    times = []
    with threadpool_limits(limits=threads):
        for s in range(n_steps):
            sl = slice(k + s * rows, k + (s + 1) * rows)
            t0 = time.perf_counter()
            orc.process_chunk(Q[sl], K[sl], V[sl], None if w.mode == "standard" else Qi)
            times.append(time.perf_counter() - t0)
    timed = times[args.warmup:]
    ms = 1e3 * sum(timed) / len(timed)
    value = rows / (ms / 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "q_heads": w.q_heads, "kv_heads": w.kv_heads, "head_dim": w.head_dim,
                       "budget_k": w.budget_k, "chunk_s": w.chunk_s, "n_instr": w.n_instr, "mode": w.mode,
                       "lm_window": w.lm_window, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                             "threads": f"BLAS pools limited to {threads} threads (threadpoolctl)"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def cpu_baseline_in_fresh_process(workload: str):
    """Times the oracle through the reference arm in a process of its own (no CUDA context, no pinned buffers, no
    sampler thread beside it), so that this figure and `--impl reference` are one measurement."""
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", workload,
           "--steps", "4", "--warmup", "1"]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        r = subprocess.run(cmd, capture_output=True, text=True, timeout=900, cwd=ROOT, env=env)
        for ln in r.stdout.splitlines():
            if ln.startswith("{"):
                d = json.loads(ln)
                cpu = d["cpu_baseline"]
                cpu["seconds_per_step"] = d["ms_per_step"] / 1e3
                cpu["steps"] = d["steps"]
                return cpu
        return {"value": None, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": "failed: " + r.stderr[-300:]}
    except Exception as e:  # noqa: BLE001
        return {"value": None, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": f"failed: {e}"}


def max_over_ranks(x: float, dist, device) -> float:
    """Whole-job time is the slowest rank's (documents are independent: no other exchange)."""
    if dist is None:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_document(w: wl.Workload, rank: int, layer: int = 0) -> wl.Document:
    """Weak scaling: rank r encodes its own document (sequence id r of the workload)."""
    return wl.make_document(w, layer=layer, seq=rank)


def rank_sequences(n_seqs: int, rank: int, world: int):
    """Ragged serving mix over several GPUs: rank r takes the sequences r, r + world, ... (no exchange between them)."""
    return list(range(rank, n_seqs, world))


# --------------------------------------------------------------------------- CUDA arm: one workload
class Job:
    """Device-resident inputs of one workload and the closure that enqueues one pass over them."""

    def __init__(self, w: wl.Workload, rank: int, world: int, doc_tokens: int = 0, sequences=None):
        from paper_2406_12018_b200.binding import Citrus
        self.w = w
        self.stream = torch.cuda.Stream()
        self.batch = w.n_seqs > 1
        self.host_docs = None
        pool = ThreadPoolExecutor(max_workers=max(1, min(8, host_cores())))
        if self.batch:
            seqs = rank_sequences(w.n_seqs, rank, world) if sequences is None else sequences
            lens = wl.sequence_lengths(w)
            if doc_tokens:
                lens = [min(x, doc_tokens) for x in lens]
            self.seqs, self.lens = seqs, [lens[s] for s in seqs]
            docs = list(pool.map(lambda s: wl.make_document(w, seq=s, n_tokens=lens[s]), seqs))
            self.tokens = sum(self.lens)
            self.sizes = [sz for n in self.lens for sz in step_sizes(w, n)]
            self.ctx = Citrus(1, w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.chunk_s, mode=w.mode, dtype=w.dtype,
                              lm_window=w.lm_window, layerwise=w.layerwise, position_shift=w.position_shift,
                              n_seqs=len(seqs))
            self.steps = []
            for c in range(-(-max(self.lens) // w.chunk_s)):
                act = [i for i, n in enumerate(self.lens) if c * w.chunk_s < n]
                sl = [slice(c * w.chunk_s, min(self.lens[i], (c + 1) * w.chunk_s)) for i in act]
                tok = [0]
                for x in sl:
                    tok.append(tok[-1] + (x.stop - x.start))
                Q, K, V = (torch.cat([getattr(docs[i], nm)[x] for i, x in zip(act, sl)]).cuda() for nm in ("Q", "K", "V"))
                Qi = torch.cat([docs[i].Q_instr for i in act]).cuda()
                ins = [w.n_instr * j for j in range(len(act) + 1)]
                self.steps.append((act, tok, Q, K, V, ins, Qi, torch.empty_like(Q)))
            self.in_bytes = sum(t.numel() * t.element_size() for st in self.steps for t in (st[2], st[3], st[4], st[7]))
            self.layers = 1
        else:
            self.layers = w.layers
            N = doc_tokens or w.doc_tokens
            docs = list(pool.map(lambda l: wl.make_document(w, layer=l, seq=rank, n_tokens=N), range(self.layers)))
            self.tokens = N
            self.sizes = step_sizes(w, N) * self.layers
            self.ctx = Citrus(self.layers, w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.chunk_s, mode=w.mode,
                              dtype=w.dtype, lm_window=w.lm_window, layerwise=w.layerwise,
                              position_shift=w.position_shift)
            self.dev = [tuple(t.cuda() for t in (d.Q, d.K, d.V, d.Q_instr)) for d in docs]
            self.out = [torch.empty_like(d[0]) for d in self.dev]
            self.in_bytes = sum(t.numel() * t.element_size() for d, o in zip(self.dev, self.out) for t in (d[0], d[1], d[2], o))
            self.host_docs = docs if self.layers == 1 else None
        pool.shutdown()
        # the inputs sit complete in HBM before anything is enqueued: the kernels may load them early
        self.ctx.set_inputs_ready(True)
        if ATTENTION_BESIDE is not None:
            self.ctx.set_attention_beside(ATTENTION_BESIDE)
        if self.batch and BATCH_LANES:
            self.ctx.set_batch_lanes(BATCH_LANES)

    def one_pass(self):
        """Every chunk of every (layer | sequence) once, in the order a model would submit them."""
        w, ctx, st = self.w, self.ctx, self.stream
        ctx.reset()
        if self.batch:
            for act, tok, Q, K, V, ins, Qi, out in self.steps:
                ctx.process_chunk_batch(0, act, tok, Q, K, V, ins, Qi, out=out, stream=st)
            return
        bounds = chunk_bounds(self.tokens, w.chunk_s)
        for ci, (a, b) in enumerate(bounds):
            for layer in range(self.layers):
                Q, K, V, Qi = self.dev[layer]
                with_instr = w.mode != "standard" or ci == len(bounds) - 1
                ctx.process_chunk(layer, Q[a:b], K[a:b], V[a:b], Qi if with_instr else None, out=self.out[layer][a:b], stream=st)

    def close(self):
        self.ctx.close()


def time_job(job: Job, steps: int, warmup: int, replays: int, use_graph: bool, dist=None, sampler=None):
    """Device time of `steps` steps of `replays` passes each; returns (ms per step, clocks, replays used)."""
    st = job.stream
    with torch.cuda.stream(st):
        for _ in range(2):
            job.one_pass()                                   # also performs every one-time set-up before capture
    torch.cuda.synchronize()
    graph = None
    if use_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            job.one_pass()
        torch.cuda.synchronize()

    def one():
        if graph is not None:
            graph.replay()
        else:
            job.one_pass()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(st):
        if replays <= 0:
            # size a step so that the timed region lasts about TARGET_TIMED_SECONDS
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for _ in range(3):
                one()
            e1.record(st)
            torch.cuda.synchronize()
            t_pass = e0.elapsed_time(e1) / 3e3
            replays = max(1, min(4096, math.ceil(TARGET_TIMED_SECONDS / (steps * t_pass))))
            replays = int(max_over_ranks(float(replays), dist, "cuda"))
        if sampler is not None:
            sampler.start()
            sampler.wait_first_sample()
        for _ in range(warmup * replays):
            one()
        barrier()
        t_begin = time.time()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(st)
        for _ in range(steps * replays):
            one()
        ev1.record(st)
        barrier()
        clocks = sampler.stop(t_begin, time.time()) if sampler is not None else None
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
    return ms_total / steps, clocks, replays, graph is not None


def kernel_figures(job: Job, passes: int, peaks):
    """The same passes again with every launch bracketed by CUDA events on the launch stream: time and share per
    kernel, a1 TFLOP/s, a3 / a4 GB/s."""
    ctx = job.ctx
    ctx.profile(True)
    with torch.cuda.stream(job.stream):
        for _ in range(passes):
            job.one_pass()
    prof = ctx.profile_read()
    ctx.profile(False)
    work = algorithmic_work(job.w, job.sizes)
    total_ms = sum(v[0] for v in prof.values()) or 1.0
    kernels = {}
    for name, (ms, cnt) in prof.items():
        if cnt:
            kernels[name] = {"us_per_launch": 1e3 * ms / cnt, "launches_per_pass": cnt // passes, "share": ms / total_ms}
    fig = {"kernels": kernels, "launches_per_pass": sum(v[1] for v in prof.values()) // passes}
    if "attention" in kernels and job.w.dtype == "bf16":
        tf = work["a1_flops"] * passes / (prof["attention"][0] / 1e3) / 1e12
        kernels["attention"]["note"] = "one launch: a1 plus the log-sum-exp pass of a2-I; flops counted: a1 only"
        fig["a1_tflops"] = tf
        fig["a1_frac_of_bf16_peak"] = tf / peaks["bf16_tflops"]
        if peaks["bf16_tflops_sustained"]:
            fig["a1_frac_of_sustained"] = tf / peaks["bf16_tflops_sustained"]
    if "select" in kernels:                                  # a3 and a4 as separate launches
        fig["a3_gbs"] = work["a3_bytes"] * passes / (prof["select"][0] / 1e3) / 1e9
        fig["a4_gbs"] = work["a4_bytes"] * passes / (prof["compact"][0] / 1e3) / 1e9
        fig["a4_frac_of_hbm_peak"] = fig["a4_gbs"] / peaks["hbm_gbs"]
        fig["a3_frac_of_hbm_peak"] = fig["a3_gbs"] / peaks["hbm_gbs"]
        kernels["compact"]["mb_per_launch"] = work["a4_bytes"] / max(1, kernels["compact"]["launches_per_pass"]) / 1e6
    elif "compact" in kernels:                               # one launch does a3 and a4
        kernels["compact"]["note"] = "one launch: a3 select + a4 compaction"
        fig["a3_a4_gbs"] = (work["a3_bytes"] + work["a4_bytes"]) * passes / (prof["compact"][0] / 1e3) / 1e9
        fig["a3_a4_frac_of_hbm_peak"] = fig["a3_a4_gbs"] / peaks["hbm_gbs"]
        kernels["compact"]["mb_per_launch"] = (work["a3_bytes"] + work["a4_bytes"]) / max(1, kernels["compact"]["launches_per_pass"]) / 1e6
    return fig, prof, work


def describe(w: wl.Workload, job: Job):
    d = {"workload": w.name, "q_heads": w.q_heads, "kv_heads": w.kv_heads, "head_dim": w.head_dim, "budget_k": w.budget_k,
         "chunk_s": w.chunk_s, "n_instr": w.n_instr, "mode": w.mode, "lm_window": w.lm_window, "dtype": w.dtype}
    if job.batch:
        d.update(sequences=len(job.lens), tokens=job.tokens, call="citrus_process_chunk_batch (sequences advance in lock step)")
    else:
        d.update(layers=job.layers, doc_tokens=job.tokens)
    if w.layerwise:
        d["granularity"] = "layer-wise"
    if w.position_shift:
        d["position_shift"] = True
    return d


def measure_config(name: str, steps: int, warmup: int, peaks, doc_tokens: int = 0):
    """One entry of the `configs` array: a short measurement of a named workload on this GPU."""
    w = ALL_WORKLOADS[name]
    t0 = time.time()
    job = Job(w, 0, 1, doc_tokens=doc_tokens)
    ms, _, replays, graphed = time_job(job, steps, warmup, 0 if name != "tiny_fp32" else 50, True)
    ms_pass = ms / replays
    fig, _, _ = kernel_figures(job, 2, peaks)
    assert job.ctx.poll_status() == 0, "a bounded device wait expired during the benchmark"
    entry = describe(w, job)
    layer_docs = job.layers if not job.batch else 1
    entry.update(ms_per_pass=ms_pass, replays_per_step=replays, steps=steps,
                 tokens_per_s=job.tokens * layer_docs / (ms_pass / 1e3))
    if layer_docs > 1:
        entry["tokens_per_s_whole_stack"] = job.tokens / (ms_pass / 1e3)
        entry["note"] = "tokens_per_s counts every layer's document (per layer); the stack figure is one document through all layers"
    entry.update({k: v for k, v in fig.items() if k != "kernels"})
    entry["kernels"] = fig["kernels"]
    entry["setup_seconds"] = round(time.time() - t0, 1)
    job.close()
    del job
    torch.cuda.empty_cache()
    return entry


# --------------------------------------------------------------------------- CUDA arm: the headline line
def run_ours(args, rank, world, local_rank):
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = ALL_WORKLOADS[args.workload]
    peaks = measured_peaks()
    job = Job(w, rank, world, doc_tokens=args.doc_tokens)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms_per_step, clocks, replays, graphed = time_job(job, args.steps, args.warmup, args.replays, not args.no_graph, dist, sampler)
    layer_docs = job.layers if not job.batch else 1
    tokens_per_pass = job.tokens * layer_docs
    if dist is not None:                                     # ragged batches: ranks hold different token counts
        t = torch.tensor([float(tokens_per_pass)], dtype=torch.float64, device="cuda")
        dist.all_reduce(t)
        total_tokens = float(t.item())
    else:
        total_tokens = float(tokens_per_pass)
    value = total_tokens * replays / (ms_per_step / 1e3)
    assert job.ctx.poll_status() == 0, "a bounded device wait expired during the benchmark"

    fig, prof, work = kernel_figures(job, 2, peaks)
    roofline = None
    if "a1_tflops" in fig:
        n_attn = prof["attention"][1] // 2
        roofline = {"bound": "tensor", "kernel": "attn_lse_kernel (a1 flops only; the launch also runs the log-sum-exp pass of a2-I)",
                    "achieved": fig["a1_tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": fig["a1_frac_of_bf16_peak"],
                    "peak_source": f"{peaks['source']} burst bf16",
                    "frac_of_sustained": fig.get("a1_frac_of_sustained"),
                    "flops_per_launch": work["a1_flops"] / max(1, n_attn),
                    "traffic": args.traffic if (args.workload == WORKLOAD and not args.doc_tokens) else None,
                    "timing": "2 of the same passes repeated with per-launch CUDA events on the launch stream",
                    "hbm_peak_gbs": peaks["hbm_gbs"],
                    **{k: v for k, v in fig.items() if k.startswith("a3") or k.startswith("a4")},
                    "kernels": fig["kernels"]}

    # ---- end to end through the host-buffer ABI call (pinned host memory, copies inside the timed region)
    e2e = None
    if job.host_docs is not None and w.mode != "standard":
        doc = job.host_docs[0]
        Qh, Kh, Vh, Qih = (t.pin_memory() for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
        outh = torch.empty_like(doc.Q).pin_memory()

        def one_document_host():
            job.ctx.reset()
            job.ctx.process_document_host(0, Qh, Kh, Vh, Qih, outh, stream=job.stream)

        e2e_steps = max(1, min(args.steps, 5))
        one_document_host()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            one_document_host()
        torch.cuda.synchronize()
        e2e_s = max_over_ranks(time.perf_counter() - t0, dist, "cuda")
        h2d = sum(t.numel() * t.element_size() for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
        d2h = doc.Q.numel() * doc.Q.element_size()
        e2e = {"value": world * job.tokens * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e2e_steps, "step": "one document",
               "api": "citrus_process_document_host"}
        del Qh, Kh, Vh, Qih, outh
    launches_per_pass = fig["launches_per_pass"]
    config = describe(w, job)
    config.update(parallelism=f"{world} GPUs, one document each, no exchange" if world > 1 else "1 GPU",
                  launch="cuda_graph" if graphed else "stream", replays_per_step=replays,
                  step=f"{replays} passes of the whole document through a1-a4",
                  inputs="resident in HBM, declared complete (citrus_set_inputs_ready)",
                  l2=f"inputs larger than L2: {job.in_bytes / 1e6:.0f} MB of Q/K/V/out per pass")
    job.close()
    del job
    torch.cuda.empty_cache()

    configs = None
    if rank == 0 and world == 1 and args.configs == "all":
        configs = []
        for name in ("tiny_fp32", "mistral7b_layer", "llama2_7b_stack", "serving_mix", "long_doc_stress"):
            try:
                configs.append(measure_config(name, 5, 3, peaks))
            except Exception as e:  # noqa: BLE001
                configs.append({"workload": name, "error": repr(e)[:300]})
        for name in args.also:
            try:
                configs.append(measure_config(name, 5, 3, peaks))
            except Exception as e:  # noqa: BLE001
                configs.append({"workload": name, "error": repr(e)[:300]})

    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        cpu = cpu_baseline_in_fresh_process(args.workload)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": w.dtype, "data": "synthetic", "config": config,
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_pass * replays * args.steps,
                "roofline": roofline, "cpu_baseline": cpu}
        if configs is not None:
            line["configs"] = configs
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_batch(args, local_rank):
    """Side measurement (not the headline): `--sequences N` documents of the workload advance together, one chunk
    each per step, through the packed ragged-batch call; `--lanes` as in citrus_set_batch_lanes (0 = chosen per call).
    Prints a reduced JSON line: whole-batch tokens/s from a CUDA graph of the run, inputs resident in HBM."""
    torch.cuda.set_device(local_rank)
    w = ALL_WORKLOADS[args.workload]
    n_tok = args.doc_tokens or w.doc_tokens
    w = wl.scaled(w, doc_tokens=n_tok, n_seqs=args.sequences, min_tokens=0)
    job = Job(w, 0, 1)
    job.ctx.set_batch_lanes(args.lanes)
    ms, clocks, replays, _ = time_job(job, max(1, min(args.steps, 200)), args.warmup, 1, True, None, ClockSampler(local_rank))
    assert job.ctx.poll_status() == 0, "a bounded device wait expired during the benchmark"
    print(json.dumps({"metric": METRIC + " (batch of sequences, side measurement)", "value": job.tokens / (ms / 1e3),
                      "unit": UNIT, "n_gpus": 1, "steps": max(1, min(args.steps, 200)), "warmup": args.warmup, "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": args.workload, "sequences": args.sequences, "doc_tokens": n_tok,
                                 "lanes": args.lanes, "budget_k": w.budget_k, "chunk_s": w.chunk_s, "mode": w.mode,
                                 "launch": "cuda_graph"},
                      "clocks": clocks}), flush=True)
    job.close()


def respawn_under_torchrun(args) -> int:
    """`--gpus N` without a launcher: start N ranks of this script on this node (one process per GPU)."""
    port = 29500 + (os.getpid() % 2000)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD, choices=sorted(ALL_WORKLOADS),
                    help="the named workload of the headline line")
    ap.add_argument("--replays", type=int, default=0,
                    help="passes of the document per step (0: as many as make the timed region last about two seconds)")
    ap.add_argument("--configs", default="all", choices=["all", "none"],
                    help="also measure the five named configurations and report them in a `configs` array (1 GPU only)")
    ap.add_argument("--also", nargs="*", default=["mistral7b_standard", "mistral7b_layerwise", "paper_mistral7b", "paper_mistral7b_shift"],
                    help="further named workloads appended to the `configs` array")
    ap.add_argument("--doc-tokens", type=int, default=0, help="truncate / set the document length")
    ap.add_argument("--no-graph", action="store_true", help="launch every chunk from the host instead of a CUDA graph")
    ap.add_argument("--skip-cpu", action="store_true", help="do not time the oracle (profiling runs)")
    ap.add_argument("--dry-run", action="store_true",
                    help="stop after the rank set-up (prints rank, world size and this rank's share of the work)")
    ap.add_argument("--sequences", type=int, default=1,
                    help="side measurement: this many documents advance together through the ragged-batch call (1 GPU)")
    ap.add_argument("--lanes", type=int, default=0, help="batch workloads and --sequences: citrus_set_batch_lanes (0 = the library's choice: one grid over all sequences)")
    ap.add_argument("--attention-beside", type=int, default=None,
                    help="largest step (attention items) whose a1 runs beside the scoring chain (citrus_set_attention_beside; 0 = off; default: the library's)")
    ap.add_argument("--traffic", type=float, default=ATTN_DRAM_TRAFFIC_BYTES,
                    help="DRAM bytes per attention launch from the committed ncu summary (null if stale)")
    args = ap.parse_args()
    global ATTENTION_BESIDE, BATCH_LANES
    ATTENTION_BESIDE = args.attention_beside
    BATCH_LANES = args.lanes
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        raise SystemExit(respawn_under_torchrun(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.dry_run:
        w = ALL_WORKLOADS[args.workload]
        share = rank_sequences(w.n_seqs, rank, world) if w.n_seqs > 1 else [rank]
        print(json.dumps({"dry_run": True, "rank": rank, "n_gpus": world, "workload": args.workload,
                          "sequences_of_this_rank": share}), flush=True)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    if args.sequences > 1:
        if world > 1:
            raise SystemExit("--sequences is a single-GPU side measurement")
        run_batch(args, local_rank)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
