#!/usr/bin/env python
"""Benchmark of the chunked instruction-aware eviction hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one whole synthetic document of the Mistral-7B-layer workload
(16384 tokens = 32 chunks of 512; 32/8 heads, head_dim 128, budget 768,
64 instruction queries, bf16, shared cache) pushed through a1-a4, chunk by chunk.
Prints ONE JSON line: document tokens/s (device-timed, inputs resident in HBM),
the same metric end to end through the host-buffer ABI call, the roofline of the
attention kernel, and the fp64 oracle timed on the host cores.
With N > 1 (torchrun) every rank runs its own document: weak scaling, no
data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2406_12018_b200 import workloads as wl  # noqa: E402

WORKLOAD = "mistral7b_layer"
# dram__bytes_read.sum + dram__bytes_write.sum of one steady-state attn_lse_kernel launch, from
# profiles/attn_lse_kernel_mistral7b_layer.md; set to None whenever that kernel changes after the capture.
ATTN_DRAM_TRAFFIC_BYTES = 10.07e6
METRIC = "document tokens/s through chunked eviction per layer"
UNIT = "tokens/s"


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
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
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
            for nm, v in zip(names, parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def attention_flops(w: wl.Workload, N: int):
    """Algorithmic flops of a1 over a document, chunk by chunk: 4 D H_q (L m + L (L+1)/2)."""
    total, per_launch, seen = 0.0, [], 0
    for s in range(0, N, w.chunk_s):
        L = min(w.chunk_s, N - s)
        m = min(w.budget_k, seen)
        f = 4.0 * w.head_dim * w.q_heads * (L * m + L * (L + 1) / 2.0)
        per_launch.append(f); total += f; seen += L
    return total, per_launch


# --------------------------------------------------------------------------- oracle arm
def oracle_tokens_per_s(w: wl.Workload, doc: wl.Document, n_chunks: int, repeats: int = 1):
    """Time the fp64 oracle, as it stands, on steady-state chunks of the workload."""
    import oracle
    orc = oracle.CitrusOracle(w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.mode, lm_window=(w.lm_window or None))
    Q, K, V, Qi = (wl.to_f64(t) for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
    fill = -(-w.budget_k // w.chunk_s)                       # chunks needed to fill the cache (untimed)
    for c in range(fill):
        sl = slice(c * w.chunk_s, (c + 1) * w.chunk_s)
        orc.process_chunk(Q[sl], K[sl], V[sl], Qi)
    times = []
    c = fill
    for _ in range(repeats):
        t0 = time.perf_counter()
        for _ in range(n_chunks):
            sl = slice(c * w.chunk_s, (c + 1) * w.chunk_s)
            orc.process_chunk(Q[sl], K[sl], V[sl], Qi)
            c += 1
        times.append(time.perf_counter() - t0)
    return n_chunks * w.chunk_s, times


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count()


def run_reference(args, rank):
    if rank != 0:
        return
    w = wl.CONFIGS[WORKLOAD]
    chunks_per_step = 2
    need = (-(-w.budget_k // w.chunk_s) + chunks_per_step * (args.steps + args.warmup)) * w.chunk_s
    doc = wl.make_document(w, n_tokens=min(w.doc_tokens, need))
    tokens, times = oracle_tokens_per_s(w, doc, chunks_per_step, repeats=args.steps + args.warmup)
    timed = times[args.warmup:]
    ms = 1e3 * sum(timed) / len(timed)
    value = tokens / (ms / 1e3)
    sample = f"{chunks_per_step} steady-state chunks ({tokens} tokens) per step after an untimed cache fill"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "q_heads": w.q_heads, "kv_heads": w.kv_heads, "head_dim": w.head_dim,
                       "budget_k": w.budget_k, "chunk_s": w.chunk_s, "n_instr": w.n_instr, "mode": w.mode,
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def max_over_ranks(x: float, dist, device) -> float:
    """Whole-job time is the slowest rank's (documents are independent: no other exchange)."""
    if dist is None:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_document(w: wl.Workload, rank: int) -> wl.Document:
    """Weak scaling: rank r encodes its own document (sequence id r of the workload)."""
    return wl.make_document(w, seq=rank)


# --------------------------------------------------------------------------- CUDA arm
def run_ours(args, rank, world, local_rank):
    from paper_2406_12018_b200.binding import Citrus
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = {**wl.CONFIGS, **wl.PAPER_SHAPES}[args.workload]
    if args.doc_tokens:
        w = wl.scaled(w, doc_tokens=args.doc_tokens, n_seqs=1, min_tokens=0)
    doc = rank_document(w, rank)
    N = doc.Q.shape[0]
    n_chunks = -(-N // w.chunk_s)
    Q, K, V, Qi = doc.Q.cuda(), doc.K.cuda(), doc.V.cuda(), doc.Q_instr.cuda()
    out = torch.empty_like(Q)
    ctx = Citrus(1, w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.chunk_s, mode=w.mode, dtype=w.dtype,
                 lm_window=w.lm_window, position_shift=w.position_shift)
    stream = torch.cuda.Stream()

    def one_document():
        ctx.reset()
        for c in range(n_chunks):
            sl = slice(c * w.chunk_s, min(N, (c + 1) * w.chunk_s))
            ctx.process_chunk(0, Q[sl], K[sl], V[sl], Qi, out=out[sl], stream=stream)

    # warm-up (also performs every one-time attribute set-up before capture)
    with torch.cuda.stream(stream):
        for _ in range(max(1, args.warmup)):
            one_document()
    torch.cuda.synchronize()
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            one_document()
        torch.cuda.synchronize()

    def step():
        if graph is not None:
            graph.replay()
        else:
            one_document()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        sampler = ClockSampler(local_rank)
        if rank == 0:
            sampler.start()
            sampler.wait_first_sample()
        for _ in range(args.warmup):
            step()
        barrier()
        t_begin = time.time()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(args.steps):
            step()
        ev1.record(stream)
        barrier()
        clocks = sampler.stop(t_begin, time.time()) if rank == 0 else None
    ms_total = ev0.elapsed_time(ev1)
    ms_total = max_over_ranks(ms_total, dist, "cuda")
    ms_per_step = ms_total / args.steps
    value = world * N / (ms_per_step / 1e3)
    assert ctx.poll_status() == 0, "a bounded device wait expired during the benchmark"

    # ---- per-kernel times: the same steps again with every launch bracketed by events
    prof_steps = min(args.steps, 20)
    ctx.profile(True)
    with torch.cuda.stream(stream):
        for _ in range(prof_steps):
            one_document()
    prof = ctx.profile_read()
    ctx.profile(False)
    total_flops, _ = attention_flops(w, N)
    attn_ms, attn_n = prof["attention"]
    peaks = measured_peaks()
    achieved = total_flops * prof_steps / (attn_ms / 1e3) / 1e12
    kern_total = sum(v[0] for v in prof.values())
    launches_per_step = sum(v[1] for v in prof.values()) // prof_steps
    n_caches = 2 if w.mode == "individual" else 1
    elt = 2
    sel_bytes = sum(4.0 * (min(w.budget_k, s) + min(w.chunk_s, N - s)) * w.kv_heads + 4.0 * min(w.budget_k, s + w.chunk_s) * w.kv_heads
                    for s in range(0, N, w.chunk_s))
    cmp_bytes = sum(2.0 * 2 * min(w.budget_k, s + w.chunk_s) * w.head_dim * elt * w.kv_heads + 8.0 * min(w.budget_k, s + w.chunk_s) * w.kv_heads
                    for s in range(0, N, w.chunk_s))
    kernels = {}
    for name, (ms, cnt) in prof.items():
        if cnt:
            kernels[name] = {"us_per_launch": 1e3 * ms / cnt, "launches_per_step": cnt // prof_steps,
                             "share": ms / kern_total}
    kernels["attention"]["note"] = "one launch: a1 plus the log-sum-exp pass of a2-I"
    # a3 + a4 run as one cluster launch (recorded under "compact"): algorithmic bytes of both steps
    kernels["compact"]["note"] = "one launch: a3 select + a4 compaction"
    if "select" in kernels:       # large steps: a3 and a4 are separate launches
        kernels["compact"]["note"] = "a4 compaction"
        kernels["select"]["gbs"] = n_caches * sel_bytes * prof_steps / (prof["select"][0] / 1e3) / 1e9
        kernels["compact"]["gbs"] = n_caches * cmp_bytes * prof_steps / (prof["compact"][0] / 1e3) / 1e9
        kernels["compact"]["mb_per_launch"] = n_caches * cmp_bytes / n_chunks / 1e6
    else:
        kernels["compact"]["gbs"] = n_caches * (sel_bytes + cmp_bytes) * prof_steps / (prof["compact"][0] / 1e3) / 1e9
        kernels["compact"]["mb_per_launch"] = n_caches * (sel_bytes + cmp_bytes) / n_chunks / 1e6
    kernels["compact"]["frac_of_hbm_peak"] = kernels["compact"]["gbs"] / peaks["hbm_gbs"]
    roofline = {"bound": "tensor", "kernel": "attn_lse_kernel (a1 flops only; the launch also runs pass 1 of a2-I)", "achieved": achieved,
                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                "peak_source": f"{peaks['source']} burst bf16 (kernel launches are short and separated)",
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
                "traffic": args.traffic if (args.workload == WORKLOAD and not args.doc_tokens) else None, "timing": f"{prof_steps} of the same steps repeated with per-launch CUDA events on the launch stream",
                "hbm_peak_gbs": peaks["hbm_gbs"], "kernels": kernels}

    # ---- end to end through the host-buffer ABI call (pinned host memory, copies inside)
    Qh, Kh, Vh, Qih = (t.pin_memory() for t in (doc.Q, doc.K, doc.V, doc.Q_instr))
    outh = torch.empty_like(doc.Q).pin_memory()

    def one_document_host():
        ctx.reset()
        ctx.process_document_host(0, Qh, Kh, Vh, Qih, outh, stream=stream)

    e2e_steps = max(1, min(args.steps, 5))
    one_document_host()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        one_document_host()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, dist, "cuda")
    h2d = sum(t.numel() * t.element_size() for t in (doc.Q, doc.K, doc.V)) + doc.Q_instr.numel() * 2
    d2h = doc.Q.numel() * 2
    e2e = {"value": world * N * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "steps": e2e_steps, "api": "citrus_process_document_host"}

    cpu = None
    if rank == 0 and not args.skip_cpu:
        n_or = n_chunks - (-(-w.budget_k // w.chunk_s))      # every steady-state chunk of the document
        tokens, times = oracle_tokens_per_s(w, doc, n_or)
        sample = f"{n_or} steady-state chunks ({tokens} tokens) of this workload after an untimed cache fill"
        cpu = {"value": tokens / times[0], "unit": UNIT, "cores": host_threads(), "kind": "oracle", "sample": sample,
               "seconds": times[0]}

    if rank == 0:
        in_bytes = sum(t.numel() * t.element_size() for t in (Q, K, V, out))
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": args.workload, "q_heads": w.q_heads, "kv_heads": w.kv_heads, "head_dim": w.head_dim,
                           "budget_k": w.budget_k, "chunk_s": w.chunk_s, "doc_tokens": N, "lm_window": w.lm_window, "n_instr": w.n_instr,
                           "mode": w.mode, "parallelism": f"{world} independent documents" if world > 1 else "1 GPU",
                           "launch": "cuda_graph" if graph is not None else "stream",
                           "l2": f"inputs larger than L2: {in_bytes / 1e6:.0f} MB of Q/K/V/out per step"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "roofline": roofline, "cpu_baseline": cpu}
        print(json.dumps(line), flush=True)
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


def run_batch(args, local_rank):
    """Side measurement (not the headline): `--sequences N` documents of the workload advance together, one chunk
    each per step, through the packed ragged-batch call; `--lanes` as in citrus_set_batch_lanes (0 = chosen per call).
    Prints a reduced JSON line: whole-batch tokens/s from a CUDA graph of the run, inputs resident in HBM."""
    from paper_2406_12018_b200.binding import Citrus
    torch.cuda.set_device(local_rank)
    w = {**wl.CONFIGS, **wl.PAPER_SHAPES}[args.workload]
    n_tok = args.doc_tokens or w.doc_tokens
    w = wl.scaled(w, doc_tokens=n_tok, n_seqs=args.sequences, min_tokens=0)
    docs = [wl.make_document(w, seq=i, n_tokens=n_tok) for i in range(args.sequences)]
    steps = []
    for c in range(-(-n_tok // w.chunk_s)):
        sl = slice(c * w.chunk_s, min(n_tok, (c + 1) * w.chunk_s))
        rows = sl.stop - sl.start
        Q, K, V = (torch.cat([getattr(d, name)[sl] for d in docs]).cuda() for name in ("Q", "K", "V"))
        steps.append((list(range(args.sequences)), [rows * i for i in range(args.sequences + 1)], Q, K, V, torch.empty_like(Q)))
    Qi = torch.cat([d.Q_instr for d in docs]).cuda()
    ins = [w.n_instr * i for i in range(args.sequences + 1)]
    ctx = Citrus(1, w.q_heads, w.kv_heads, w.head_dim, w.budget_k, w.chunk_s, mode=w.mode, dtype=w.dtype,
                 lm_window=w.lm_window, position_shift=w.position_shift, n_seqs=args.sequences)
    ctx.set_batch_lanes(args.lanes)
    stream = torch.cuda.Stream()

    def all_documents():
        ctx.reset()
        for slots, tok, Q, K, V, out in steps:
            ctx.process_chunk_batch(0, slots, tok, Q, K, V, ins, Qi, out=out, stream=stream)

    with torch.cuda.stream(stream):
        for _ in range(max(1, args.warmup)):
            all_documents()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        all_documents()
    n_steps = max(1, min(args.steps, 200))
    with torch.cuda.stream(stream):
        sampler = ClockSampler(local_rank)
        sampler.start(); sampler.wait_first_sample()
        for _ in range(args.warmup):
            graph.replay()
        torch.cuda.synchronize()
        t_begin = time.time()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(n_steps):
            graph.replay()
        ev1.record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop(t_begin, time.time())
    ms = ev0.elapsed_time(ev1) / n_steps
    assert ctx.poll_status() == 0, "a bounded device wait expired during the benchmark"
    print(json.dumps({"metric": METRIC + " (batch of sequences, side measurement)", "value": args.sequences * n_tok / (ms / 1e3),
                      "unit": UNIT, "n_gpus": 1, "steps": n_steps, "warmup": args.warmup, "ms_per_step": ms,
                      "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": args.workload, "sequences": args.sequences, "doc_tokens": n_tok,
                                 "lanes": args.lanes, "budget_k": w.budget_k, "chunk_s": w.chunk_s, "mode": w.mode,
                                 "launch": "cuda_graph"},
                      "clocks": clocks}), flush=True)
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=WORKLOAD,
                    choices=[k for k, v in {**wl.CONFIGS, **wl.PAPER_SHAPES}.items() if v.dtype == "bf16"],
                    help="another named workload (layer 0, one sequence) instead of the headline one")
    ap.add_argument("--doc-tokens", type=int, default=0, help="truncate / set the document length")
    ap.add_argument("--no-graph", action="store_true", help="launch every chunk from the host instead of a CUDA graph")
    ap.add_argument("--skip-cpu", action="store_true", help="do not time the oracle (profiling runs)")
    ap.add_argument("--sequences", type=int, default=1,
                    help="side measurement: this many documents advance together through the ragged-batch call (1 GPU)")
    ap.add_argument("--lanes", type=int, default=0, help="with --sequences: side streams of the batch call (0 = automatic)")
    ap.add_argument("--traffic", type=float, default=ATTN_DRAM_TRAFFIC_BYTES,
                    help="DRAM bytes per attention launch from the committed ncu summary (null if stale)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
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
