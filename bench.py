"""Benchmark of the ASAP prune step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1..c6] [--impl reference]

A step is one pass of the whole prune step (attention mass, salience, mask, masked ranking
scores, top-k, cosine assignment, weighted merge, compaction) over one synthetic batch.  The
default workload is c4, the largest single-GPU shape: the LLaVA-NeXT AnyRes batch of 64
sequences (2880 visual tokens each, ragged text, keep 576).  One JSON line is printed by rank 0:

  value          visual tokens per second, inputs resident in HBM, all ranks together; the timed steps
                 are replayed from a CUDA graph holding one step per device copy of the inputs
                 (config.timed_as; --no-graph times directly launched steps, which the line also
                 reports as direct_launch)
  e2e            the same with inputs in pinned host memory: every step copies them to the
                 device, runs the step through the C ABI and reads the shortened batch back (the
                 copies of neighbouring steps overlap: two sets of buffers, three streams)
  roofline       the kernel with the largest share of the step, against the measured peak
  kernels        per-kernel device time (CUDA events recorded by the library on its stream), each
                 with its own roofline object
  sustained      at least a second of back-to-back steps with the SM clock sampled meanwhile
  other_workloads  short runs of c1 (rotated inputs and L2-warm), c2, c3, and the c5 schedule:
                 three successive steps 2304 -> 1152 -> 576 -> 288 on the batch of 32, Q/K re-drawn
                 at the gathered positions, value = B * 2304 / (sum of the three step times)
  cpu_baseline   the float64 CPU oracle timed on this host's cores on a few sequences

With --impl reference the CPU oracle alone is timed (rank 0 only).
With N > 1 every rank prunes its own batch of the same shape (sequences are independent, there
is no exchange step): the ranks only meet at the barriers around the timed region.  Started
without a launcher, `--gpus N` spawns the N ranks itself.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import socket
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2603_14549_b200 import replicas as R
from paper_2603_14549_b200 import workloads as W

METRIC = "visual_tokens_per_sec"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

WORKLOADS = {
    "c1": "LLaVA-1.5-7B single sequence: 35 system + 576 visual + 32 text, D=4096, 32x128 heads, keep 192",
    "c2": "LLaVA-1.5-7B batch 16: 35 system + 576 visual + text U[16,128], D=4096, 32x128 heads, keep 64",
    "c3": "LLaVA-NeXT-7B batch 8: 35 system + 2304 visual + 64 text, D=4096, 32x128 heads, keep 320",
    "c4": "LLaVA-NeXT AnyRes batch 64 (largest single-GPU configuration): 35 system + 2880 visual + text U[32,256], "
          "D=4096, 32x128 heads, keep 576",
    "c5": "13B-shaped batch 32, first step of 2304->1152: 35 system + 2304 visual + 128 text, D=5120, 40x128 heads",
    "c6": "InternVL-2.5-8B-shaped batch 8: 35 system + 1536 visual (6 tiles of 256) + 64 text, D=4096, 32x128 heads, keep 510",
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic(workload):
    """DRAM bytes per launch of each kernel from the committed ncu captures, or {}."""
    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        return json.load(f).get(workload, {})


# ------------------------------------------------------------------------------------------
# algorithmic traffic / work of each kernel for one launch over the whole batch
# ------------------------------------------------------------------------------------------
def algorithmic(batch, keep_k, rank_visual=False):
    """Bytes each kernel must move and flops it must do, from the problem sizes alone:
    every operand it consumes read once, every result written once (bf16 = 2 bytes)."""
    D = batch.D
    out = {name: {"bytes": 0, "flops": 0} for name in
           ("qsum", "mass_salience", "salience", "score", "head_sum", "select", "kept_gather", "sim", "merge_compact",
            "prepare", "role_map")}
    for b in range(batch.B):
        n = int(batch.cu_seqlens[b + 1] - batch.cu_seqlens[b])
        nv, tl = int(batch.vis_len[b]), int(batch.text_len[b])
        t0 = int(batch.text_start[b])
        row = D * 2
        out["qsum"]["bytes"] += nv * row
        out["qsum"]["flops"] += nv * D
        out["mass_salience"]["bytes"] += nv * row + nv * 12
        out["mass_salience"]["flops"] += 2 * nv * D
        out["salience"]["bytes"] += batch.H * nv * 4 + nv * 12      # per-head masses in, mass / salience / mask out
        # ranking rows = text span: queries once, every key they may attend to once
        out["score"]["bytes"] += tl * row + (t0 + tl) * row + nv * 4
        out["score"]["flops"] += 2 * tl * (t0 + (tl + 1) // 2) * D
        if rank_visual:     # image span ranked too: its rows see the prefix and, through Eq. 3, every visual key
            v0 = int(batch.vis_start[b])
            out["score"]["bytes"] += nv * row
            out["score"]["flops"] += 2 * nv * (v0 + nv) * D
        out["select"]["bytes"] += nv * 4 + nv * 4
        out["head_sum"]["bytes"] += batch.H * nv * 4 + nv * 4
        out["kept_gather"]["bytes"] += 2 * keep_k * row
        out["kept_gather"]["flops"] += 2 * keep_k * D
        out["sim"]["bytes"] += nv * row
        out["sim"]["flops"] += 2 * (nv - keep_k) * keep_k * D
        out["merge_compact"]["bytes"] += n * row + (n - nv + keep_k) * row
        out["merge_compact"]["flops"] += 2 * nv * D
    return out


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.path = tempfile.mktemp(prefix="asap_clocks_", suffix=".csv")
        self.proc = None
        self.index = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Samples taken between the wall-clock times t_begin and t_end (the timed region); if
        the region was too short to catch one, all samples of the run."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        import datetime
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 8:
                        continue
                    try:
                        ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                        rows.append((ts, float(parts[1]), float(parts[2]), float(parts[3]),
                                     [nm for nm, v in zip(names, parts[4:8]) if v.lower().startswith("active")]))
                    except ValueError:
                        continue
            os.unlink(self.path)
        except OSError:
            pass
        inside = [r for r in rows if t_begin is not None and t_begin <= r[0] <= t_end]
        use = inside if inside else rows
        reasons = sorted({nm for r in use for nm in r[4]})
        return {"sm_mhz": statistics.median(r[1] for r in use) if use else None,
                "sm_max_mhz": max(r[2] for r in use) if use else None,
                "power_w_max": max(r[3] for r in use) if use else None, "reasons": reasons,
                "samples": len(use), "samples_in_timed_region": len(inside)}


# ------------------------------------------------------------------------------------------
# CPU oracle legs (the only places that touch oracle/)
# ------------------------------------------------------------------------------------------
def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def time_oracle(batch, keep_k, budget_s=12.0, max_samples=None):
    """Runs the float64 oracle sequence by sequence until `budget_s` of CPU time is used or the
    batch is exhausted; returns (visual tokens per second, seconds, sequences, threads).  The
    oracle walks the sequences one after the other; `threads` is the size of the BLAS pool its
    matrix products may use, not a parallel-over-sequences run."""
    from oracle import asap_oracle as O
    import numpy as np

    def bits(t):   # bf16 tensor -> uint16 bit patterns, the form the oracle takes
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)
    threads = blas_threads()
    done, tokens = 0, 0
    t_start = time.perf_counter()
    limit = batch.B if max_samples is None else min(batch.B, max_samples)
    while True:
        b = done % limit          # a small batch is walked again until the time budget is used
        rows = batch.sample_rows(b)
        O.prune_sample(bits(batch.q[rows]), bits(batch.k[rows]), bits(batch.hidden[rows]),
                       batch.pos_ids[rows].numpy(), int(batch.vis_start[b]), int(batch.vis_len[b]),
                       int(batch.text_start[b]), int(batch.text_len[b]), keep_k)
        done += 1
        tokens += int(batch.vis_len[b])
        elapsed = time.perf_counter() - t_start
        if elapsed >= budget_s or (budget_s > 1e8 and done >= limit):
            break
    secs = time.perf_counter() - t_start
    return tokens / secs, secs, done, threads


CORES_NOTE = "cores = size of the BLAS thread pool the numpy oracle may use; sequences are evaluated one after the other"


def run_reference(args):
    rank, size, _ = R.world()
    if rank != 0:
        return
    batch = W.config(args.workload, B=args.ref_sequences)
    keep_k = batch.keep_k
    for _ in range(args.warmup):
        time_oracle(batch, keep_k, budget_s=1e9, max_samples=1)
    t0 = time.perf_counter()
    tokens = 0
    threads = 1
    for _ in range(args.steps):
        v, secs, done, threads = time_oracle(batch, keep_k, budget_s=1e9)
        tokens += sum(int(batch.vis_len[b]) for b in range(done))
    secs = time.perf_counter() - t0
    value = tokens / secs
    sample = f"{batch.B} sequence(s) of {args.workload} per step, float64 numpy oracle; {CORES_NOTE}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": f"{args.workload}: {WORKLOADS[args.workload]}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------------------------
# CUDA arm: one workload set up on the device
# ------------------------------------------------------------------------------------------
class Setup:
    """A batch resident on the device in `n_copies` copies (rotated so that no step finds its inputs
    in L2), a library context sized for it, and one set of outputs."""

    def __init__(self, A, batch, keep_k, device, local, stream, n_copies=None, rank_visual=False):
        self.A, self.batch, self.keep_k, self.device, self.stream = A, batch, keep_k, device, stream
        self.params = A.Params(keep_k=keep_k)
        self.units = int(batch.vis_len.sum())
        self.in_bytes = sum(t.numel() * t.element_size() for t in (batch.q, batch.k, batch.hidden, batch.pos_ids))
        self.n_copies = n_copies if n_copies else max(2, min(64, -(-(8 * L2_BYTES) // self.in_bytes)))
        self.ctx = A.asap_init(local, max_total_tokens=batch.total, max_B=batch.B, max_H=batch.H, max_D=batch.D,
                               max_keep_rows=batch.B * keep_k)
        first = A.make_inputs(batch, device)
        self.copies = [first]
        for _ in range(self.n_copies - 1):
            self.copies.append(dataclasses.replace(first, q=first.q.clone(), k=first.k.clone(),
                                                   hidden=first.hidden.clone(), pos_ids=first.pos_ids.clone()))
        if rank_visual:       # Eq. 3 acts on these rows; the score kernel becomes a dense, tensor-pipe-heavy pass
            rs = batch.vis_start.to(device)
            rl = (batch.vis_len + batch.text_len).to(device)
            self.copies = [dataclasses.replace(c, rank_start=rs, rank_len=rl,
                                               max_rank=int((batch.vis_len + batch.text_len).max()))
                           for c in self.copies]
        self.out = A.alloc_outputs(self.copies[0], keep_k)

    def step(self, i):
        self.A.asap_prune_step(self.ctx, self.copies[i % self.n_copies], self.params, self.out, self.stream)

    def l2_note(self):
        if self.n_copies == 1:
            return "one device copy of the inputs: every step after the first finds them in L2 where they fit"
        return (f"inputs rotate over {self.n_copies} device copies ({self.n_copies * self.in_bytes / 2**20:.0f} MiB) "
                f"so no step finds its inputs in the {L2_BYTES // 2**20} MiB L2")

    def free(self):
        self.A.asap_free(self.ctx)
        self.copies = None
        self.out = None


def capture_graph(S):
    """One CUDA graph holding one step per device copy (the library's calls are capturable: no
    allocation, no synchronisation, the side stream joins back inside the call)."""
    A = S.A
    c0 = A.asap_launch_count(S.ctx)
    graph = torch.cuda.CUDAGraph()
    graph.capture_begin()
    for i in range(S.n_copies):
        S.step(i)
    graph.capture_end()
    launches = A.asap_launch_count(S.ctx) - c0
    graph.replay()
    torch.cuda.synchronize()
    A.asap_check(S.ctx)
    return graph, launches


def time_steps(S, steps, warmup, use_graph=True, sync_ranks=False, sampler=None):
    """W warm-up steps, then exactly `steps` steps between two events on the launching stream."""
    A = S.A
    for i in range(warmup):
        S.step(i)
    torch.cuda.synchronize()
    A.asap_check(S.ctx)
    graph, per_replay, launches_per_replay = None, 1, 0
    if use_graph and steps % S.n_copies == 0:
        try:
            graph, launches_per_replay = capture_graph(S)
            per_replay = S.n_copies
        except Exception as ex:                      # capture not available: fall back to direct launches
            print(f"bench.py: graph capture failed ({ex!r}); timing directly launched steps", file=sys.stderr)
            graph, per_replay = None, 1
    n_marks = steps // per_replay
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_marks + 1)]
    launches0 = A.asap_launch_count(S.ctx)
    if sync_ranks:
        R.barrier()
    torch.cuda.synchronize()
    wall_begin = time.time()
    marks[0].record(S.stream)
    for i in range(n_marks):
        if graph is not None:
            graph.replay()
        else:
            S.step(warmup + i)
        marks[i + 1].record(S.stream)
    torch.cuda.synchronize()
    if sync_ranks:
        R.barrier()
    wall_end = time.time()
    clocks = sampler.stop(wall_begin, wall_end) if sampler is not None else None
    launches = launches_per_replay * n_marks if graph is not None else A.asap_launch_count(S.ctx) - launches0
    total_ms = marks[0].elapsed_time(marks[-1])
    per_step = sorted(marks[i].elapsed_time(marks[i + 1]) / per_replay for i in range(n_marks))
    A.asap_check(S.ctx)
    timed_as = (f"CUDA graph of {S.n_copies} steps (one per input copy) replayed {n_marks} times"
                if graph is not None else "directly launched steps")
    return {"total_ms": total_ms, "ms_per_step": total_ms / steps, "per_step_ms": per_step, "launches": launches,
            "timed_as": timed_as, "graph": graph, "clocks": clocks, "marks": n_marks}


def kernel_times(S, steps, first=0):
    """Per-kernel device times: the same steps with the library's own events on (in order, one stream)."""
    A = S.A
    A.asap_profile(S.ctx, True)
    for i in range(min(steps, 1000)):        # the library times at most 16384 events between reads
        S.step(first + i)
    torch.cuda.synchronize()
    kt = A.asap_profile_read(S.ctx)
    A.asap_profile(S.ctx, False)
    return kt


def kernel_table(ktimes, alg, peaks, peak_kind, traffic):
    """avg time, share and a roofline object per kernel, largest share first."""
    ksum = sum(ms for _, ms in ktimes.values()) or 1.0
    kernels = {}
    for name, (n, ms) in sorted(ktimes.items(), key=lambda kv: -kv[1][1]):
        avg_s = ms / max(n, 1) * 1e-3
        a = alg.get(name, {"bytes": 0, "flops": 0})
        gbs = a["bytes"] / avg_s / 1e9 if avg_s > 0 else 0.0
        tfs = a["flops"] / avg_s / 1e12 if avg_s > 0 else 0.0
        hbm_frac, tc_frac = gbs / peaks["hbm_gbs"], tfs / peaks["bf16_tflops"]
        if name in ("sim", "score") and tc_frac > hbm_frac:
            roof = {"bound": "tensor", "achieved": tfs, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": tc_frac, "peak_kind": peak_kind + " (burst)"}
        elif a["bytes"] > 0:
            roof = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": hbm_frac,
                    "peak_kind": peak_kind}
        else:
            roof = None
        if roof is not None:
            roof["traffic"] = traffic.get(name)
            roof["algorithmic_bytes_per_launch"] = a["bytes"]
            roof["algorithmic_flops_per_launch"] = a["flops"]
            roof["avg_launch_us"] = avg_s * 1e6
        kernels[name] = {"launches": n, "avg_us": avg_s * 1e6, "share": ms / ksum, "alg_GBs": gbs, "alg_TFLOPs": tfs,
                         "roofline": roof}
    return kernels


def dominant_roofline(kernels):
    for name, k in kernels.items():
        if k["roofline"] is not None:
            r = dict(k["roofline"])
            r["kernel"] = name
            return r
    return None


def short_run(A, name, batch, keep_k, device, local, stream, peaks, peak_kind, steps, n_copies=None):
    """A compact record of one more workload: ms per step, its kernels, the dominant kernel's roofline."""
    S = Setup(A, batch, keep_k, device, local, stream, n_copies=n_copies)
    steps = max(S.n_copies, steps // S.n_copies * S.n_copies)
    t = time_steps(S, steps, 3)
    kt = kernel_times(S, min(steps, 20))
    kernels = kernel_table(kt, algorithmic(batch, keep_k), peaks, peak_kind, load_traffic(name))
    rec = {"workload": f"{name}: {WORKLOADS[name]}", "keep_k": keep_k, "steps": steps, "ms_per_step": t["ms_per_step"],
           "visual_tokens_per_sec": S.units / (t["ms_per_step"] * 1e-3), "l2": S.l2_note(), "timed_as": t["timed_as"],
           "roofline": dominant_roofline(kernels),
           "kernel_us": {n: round(k["avg_us"], 2) for n, k in kernels.items()},
           "kernel_frac_of_roof": {n: round(k["roofline"]["frac"], 4) for n, k in kernels.items() if k["roofline"]}}
    return rec, S


def c5_schedule(A, device, local, stream, peaks, peak_kind, steps):
    """The progressive schedule: three successive prune steps 2304 -> 1152 -> 576 -> 288 on the batch of 32.
    Every step consumes the previous step's hidden states and gathered position ids; its Q / K are drawn
    afresh and rotated at those positions (on the host, outside every timed region).  Each step is timed
    on its own (inputs rotated over device copies); value = B * 2304 / (sum of the three step times)."""
    batch = W.config("c5")
    cur, recs, total_ms = batch, [], 0.0
    for step_i, k in enumerate(W.C5_SCHEDULE):
        cur.keep_k = k
        rec, S = short_run(A, "c5", cur, k, device, local, stream, peaks, peak_kind, steps)
        rec["workload"] = f"c5 step {step_i + 1}: {int(cur.vis_len[0])} -> {k} visual tokens, batch {cur.B}, D={cur.D}"
        total_ms += rec["ms_per_step"]
        recs.append(rec)
        S.step(0)
        torch.cuda.synchronize()
        ocu = S.out.out_cu_seqlens.cpu()
        n_out = int(ocu[-1])
        hidden, pos = S.out.out_hidden[:n_out].cpu(), S.out.out_pos[:n_out].cpu()
        S.free()
        if step_i + 1 < len(W.C5_SCHEDULE):
            q, kk = W.redraw_qk(pos, ocu, cur.H, cur.head_dim, cur.seed, step_i + 1)
            cur = W.Batch(name="c5", B=cur.B, H=cur.H, head_dim=cur.head_dim, D=cur.D, keep_k=k, cu_seqlens=ocu,
                          vis_start=cur.vis_start, vis_len=torch.full_like(cur.vis_len, k),
                          text_start=cur.vis_start + k, text_len=cur.text_len, q=q, k=kk, hidden=hidden,
                          pos_ids=pos, seed=cur.seed)
    units = batch.B * 2304
    return {"schedule": "2304 -> 1152 -> 576 -> 288, batch 32, D=5120, 40 heads; Q/K re-drawn per step at the gathered positions",
            "steps": recs, "sum_ms": total_ms, "visual_tokens_per_sec": units / (total_ms * 1e-3),
            "definition": "B * 2304 / (sum of the three step times)"}


def run_cuda(args):
    from paper_2603_14549_b200 import binding as A   # raises if libasap.so is missing: no fallback
    rank, size, local = R.init("nccl")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (B200); there is no CPU path")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    peaks, peak_kind = load_peaks()

    seed = R.replica_seed(W.BASE_SEED + int(args.workload[1]) - 1, rank)
    batch = W.config(args.workload, B=args.sequences, seed=seed)
    keep_k = batch.keep_k
    stream = torch.cuda.Stream(device=device)     # a stream of our own: the legacy stream cannot be captured
    torch.cuda.set_stream(stream)
    rank_visual = args.rank_rows == "visual+text"
    S = Setup(A, batch, keep_k, device, local, stream, rank_visual=rank_visual)
    ctx, copies, out, params, n_copies, units = S.ctx, S.copies, S.out, S.params, S.n_copies, S.units

    # ---- device-resident timing (the headline): K steps replayed from a graph of one step per input copy
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    t = time_steps(S, args.steps, args.warmup, use_graph=not args.no_graph, sync_ranks=True,
                   sampler=sampler if rank == 0 else None)
    clocks, graph = t["clocks"], t["graph"]
    total_ms_max = R.max_over_ranks(t["total_ms"], device)
    units_all = R.sum_over_ranks(units, device)
    per_step = t["per_step_ms"]
    solo = size == 1            # the legs below describe one GPU; with replicas only the headline and e2e run

    # ---- sustained: at least a second of back-to-back steps, SM clock sampled meanwhile
    sustained = None
    if solo and graph is not None and args.sustained_s > 0:
        n_rep = max(1, int(args.sustained_s * 1e3 / (t["ms_per_step"] * n_copies)) + 1)
        smp = ClockSampler(local)
        smp.start()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        w0 = time.time()
        s0.record(stream)
        for _ in range(n_rep):
            graph.replay()
        s1.record(stream)
        torch.cuda.synchronize()
        w1 = time.time()
        sc = smp.stop(w0, w1)
        ms = s0.elapsed_time(s1) / (n_rep * n_copies)
        sustained = {"steps": n_rep * n_copies, "seconds": s0.elapsed_time(s1) * 1e-3, "ms_per_step": ms,
                     "value": units / (ms * 1e-3), "unit": UNIT, "clocks": sc,
                     "ms_times_mhz": ms * sc["sm_mhz"] if sc.get("sm_mhz") else None,
                     "headline_ms_times_mhz": (t["ms_per_step"] * clocks["sm_mhz"]
                                               if clocks and clocks.get("sm_mhz") else None)}
        A.asap_check(ctx)

    # ---- per-kernel device times: the same steps again with the library's own events on
    ktimes = kernel_times(S, min(args.steps, 50), args.warmup)

    # ---- the same steps launched directly through the API, reported beside the headline
    direct = None
    if solo and graph is not None and args.direct_steps > 0:
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(3):
            S.step(i)
        torch.cuda.synchronize()
        d0.record(stream)
        for i in range(args.direct_steps):
            S.step(i)
        d1.record(stream)
        torch.cuda.synchronize()
        direct = {"us_per_step": d0.elapsed_time(d1) / args.direct_steps * 1e3, "steps": args.direct_steps}

    # ---- KV-cache compaction of the layers up to the pruning layer (next-row feature, timed apart
    # from the step: keys and values of `kv_layers` layers gathered with the step's row map)
    kv = None
    if solo and args.kv_layers > 0:
        n_out = batch.total - units + batch.B * keep_k
        n_t = 2 * args.kv_layers
        kv_src = [torch.randn(batch.total, batch.D, device=device).to(torch.bfloat16) for _ in range(n_t)]
        kv_dst = [torch.empty(out.out_hidden.shape[0], batch.D, dtype=torch.bfloat16, device=device) for _ in range(n_t)]
        n_rows = out.out_cu_seqlens[batch.B:]
        for _ in range(3):
            A.asap_compact_kv(ctx, out.src_row, n_rows, kv_src, kv_dst, stream)
        k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        k0.record(stream)
        for _ in range(20):
            A.asap_compact_kv(ctx, out.src_row, n_rows, kv_src, kv_dst, stream)
        k1.record(stream)
        torch.cuda.synchronize()
        kv_us = k0.elapsed_time(k1) / 20 * 1e3
        kv_bytes = 2 * n_out * batch.D * 2 * n_t
        from paper_2603_14549_b200 import flops as F
        kv = {"layers": args.kv_layers, "tensors": n_t, "rows_out": n_out, "bytes": kv_bytes, "us": kv_us,
              "GBs": kv_bytes / kv_us / 1e3, "frac_of_hbm_peak": kv_bytes / kv_us / 1e3 / peaks["hbm_gbs"],
              "roofline": {"kernel": "gather_rows", "bound": "hbm", "achieved": kv_bytes / kv_us / 1e3,
                           "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": kv_bytes / kv_us / 1e3 / peaks["hbm_gbs"],
                           "traffic": (load_traffic(args.workload).get("gather_rows_per_tensor") or 0) * n_t or None,
                           "peak_kind": peak_kind},
              "storage": F.kv_storage_bytes(batch.total, n_out, args.kv_layers, batch.D)}
        del kv_src, kv_dst

    # ---- the three stages called one by one (asap_score / asap_select / asap_merge, and the score with one
    # mask per head): the kernels only these entry points launch (head_sum, prepare, role_map, mass_heads)
    staged = None
    if solo and args.staged_iters > 0:
        out_h = A.alloc_outputs(copies[0], keep_k, per_head=True) if batch.H % 2 == 0 else None
        p_h = dataclasses.replace(params, per_head_mask=True)
        sal, kidx, didx, rsc = (x.clone() for x in (out.salience, out.keep_idx, out.drop_idx, out.rank_score))

        def staged_call(i):
            c = copies[i % n_copies]
            A.asap_score(ctx, c, params, out, stream)
            A.asap_select(ctx, c, params, rsc, out, stream)
            A.asap_merge(ctx, c, params, sal, kidx, didx, out, stream)
            if out_h is not None:
                A.asap_score(ctx, c, p_h, out_h, stream)
        for i in range(2):
            staged_call(i)
        torch.cuda.synchronize()
        A.asap_check(ctx)
        A.asap_profile(ctx, True)
        for i in range(args.staged_iters):
            staged_call(i)
        torch.cuda.synchronize()
        sk = {name: ms / max(n, 1) * 1e3 for name, (n, ms) in A.asap_profile_read(ctx).items()}
        A.asap_profile(ctx, False)
        hs_bytes = sum(batch.H * int(v) * 4 + int(v) * 4 for v in batch.vis_len)
        mh_bytes = sum(int(v) * batch.D * 2 + 2 * batch.H * int(v) * 4 for v in batch.vis_len)
        staged = {"calls": "asap_score, asap_select, asap_merge, asap_score(per_head_mask)", "kernel_us": sk,
                  "head_sum_GBs": hs_bytes / sk["head_sum"] / 1e3 if sk.get("head_sum") else None,
                  "mass_heads_GBs": mh_bytes / sk["mass_heads"] / 1e3 if sk.get("mass_heads") else None}
        A.asap_prune_step(ctx, copies[0], params, out, stream)     # the later legs use the step's own results
        torch.cuda.synchronize()
        del out_h

    # ---- stage 2 as Sec. 4.2 words it (routing inside the kept set, refill by attention mass), timed
    # apart from the step on the step's own stage-1 results
    cons = None
    if solo and args.consolidate_iters > 0 and keep_k < int(batch.vis_len.max()):
        p2 = dataclasses.replace(params, sim_threshold=args.consolidate_threshold)
        st1 = [x.clone() for x in (out.mass, out.salience, out.keep_idx, out.drop_idx)]
        out2 = A.alloc_outputs(copies[0], keep_k)
        scratch = torch.empty(A.asap_consolidate_scratch_bytes(batch.B, keep_k), dtype=torch.uint8, device=device)
        n_abs = torch.zeros(batch.B, dtype=torch.int32, device=device)
        call = lambda i: A.asap_consolidate(ctx, copies[i % n_copies], p2, st1[0], st1[1], st1[2], st1[3], scratch,
                                            out2, n_abs, stream)
        for i in range(3):
            call(i)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        c0.record(stream)
        for i in range(args.consolidate_iters):
            call(i)
        c1.record(stream)
        torch.cuda.synchronize()
        A.asap_check(ctx)
        A.asap_profile(ctx, True)
        for i in range(args.consolidate_iters):
            call(i)
        torch.cuda.synchronize()
        ck = {name: ms / max(n, 1) * 1e3 for name, (n, ms) in A.asap_profile_read(ctx).items()}
        A.asap_profile(ctx, False)
        cons = {"threshold": args.consolidate_threshold, "us": c0.elapsed_time(c1) / args.consolidate_iters * 1e3,
                "absorbed_per_sequence": float(n_abs.float().mean()), "kernel_us": ck}
        del scratch, out2

    # ---- the layer's attention under the SG-BiMask (Eq. 4 applied to the values), timed apart from the
    # step with the step's own mask vector
    attn = None
    if solo and args.attention_iters > 0:
        v_dev = W.draw_values(batch, 4242).to(device)
        a_out = torch.empty_like(v_dev)
        a_scr = torch.empty(A.asap_attention_scratch_bytes(batch.total, batch.D), dtype=torch.uint8, device=device)
        acall = lambda i: A.asap_attention(ctx, copies[i % n_copies], params, out.mask_log, v_dev, a_scr, a_out, stream)
        for i in range(2):
            acall(i)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a0.record(stream)
        for i in range(args.attention_iters):
            acall(i)
        a1.record(stream)
        torch.cuda.synchronize()
        A.asap_check(ctx)
        A.asap_profile(ctx, True)
        for i in range(min(args.attention_iters, 10)):
            acall(i)
        torch.cuda.synchronize()
        ak = {name: ms / max(n, 1) * 1e3 for name, (n, ms) in A.asap_profile_read(ctx).items()}
        A.asap_profile(ctx, False)
        # admitted (query, key) pairs: the causal triangle plus, for rows of the image span, the later keys of the span
        pairs = 0
        for b_ in range(batch.B):
            n_, nv_ = int(batch.cu_seqlens[b_ + 1] - batch.cu_seqlens[b_]), int(batch.vis_len[b_])
            pairs += n_ * (n_ + 1) // 2 + nv_ * (nv_ - 1) // 2
        a_us = a0.elapsed_time(a1) / args.attention_iters * 1e3
        a_flops = 4.0 * batch.head_dim * pairs * batch.H
        attn = {"us": a_us, "admitted_pairs": pairs, "flops": a_flops, "TFLOPs": a_flops / a_us / 1e6,
                "frac_of_bf16_peak": a_flops / a_us / 1e6 / peaks["bf16_tflops"], "kernel_us": ak}
        if ak.get("attention"):       # the attention kernel alone against the measured burst peak
            attn["roofline"] = {"kernel": "attention", "bound": "tensor", "achieved": a_flops / ak["attention"] / 1e6,
                                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                "frac": a_flops / ak["attention"] / 1e6 / peaks["bf16_tflops"], "traffic": None,
                                "peak_kind": peak_kind + " (burst)"}
        del v_dev, a_out, a_scr

    # ---- end to end from pinned host memory: every step copies its inputs to the device, runs the
    # step through the C ABI and reads the shortened batch back; the three legs run on streams of their
    # own over two sets of buffers, so the copies of neighbouring steps overlap (PCIe is full duplex),
    # and the host waits for a step's results before it lets the step two later reuse their buffers
    e2e = None
    if not args.no_e2e:
        host = {n: getattr(batch, n).contiguous().pin_memory() for n in ("q", "k", "hidden", "pos_ids")}
        n_out_rows = batch.total - units + batch.B * keep_k
        dev_in = [copies[0], copies[1 % n_copies]]
        dev_out = [out, A.alloc_outputs(copies[0], keep_k)]
        host_out = [{"out_hidden": torch.empty(n_out_rows, batch.D, dtype=torch.bfloat16).pin_memory(),
                     "out_pos": torch.empty(n_out_rows, dtype=torch.int32).pin_memory(),
                     "out_cu_seqlens": torch.empty(batch.B + 1, dtype=torch.int32).pin_memory(),
                     "keep_idx": torch.empty(batch.B, keep_k, dtype=torch.int32).pin_memory()} for _ in range(2)]
        h2d = sum(x.numel() * x.element_size() for x in host.values())
        d2h = sum(x.numel() * x.element_size() for x in host_out[0].values())
        s_in, s_out = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_run = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def e2e_steps(n, first, last):
            first.record(s_in)
            for i in range(n):
                j = i & 1
                if i >= 2:
                    ev_out[j].synchronize()          # the caller has step i - 2's results before its buffers go round
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_run[j])   # step i - 2 no longer reads these inputs
                    for name, x in host.items():
                        getattr(dev_in[j], name).copy_(x, non_blocking=True)
                    ev_in[j].record(s_in)
                stream.wait_event(ev_in[j])
                A.asap_prune_step(ctx, dev_in[j], params, dev_out[j], stream)
                ev_run[j].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_run[j])
                    o = dev_out[j]
                    host_out[j]["out_hidden"].copy_(o.out_hidden[:n_out_rows], non_blocking=True)
                    host_out[j]["out_pos"].copy_(o.out_pos[:n_out_rows], non_blocking=True)
                    host_out[j]["out_cu_seqlens"].copy_(o.out_cu_seqlens, non_blocking=True)
                    host_out[j]["keep_idx"].copy_(o.keep_idx, non_blocking=True)
                    ev_out[j].record(s_out)
            s_out.synchronize()
            last.record(s_out)
            last.synchronize()

        e_steps = max(4, min(args.steps, args.e2e_steps))
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_steps(4, w0, w1)
        R.barrier(); torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_steps(e_steps, e0, e1)
        torch.cuda.synchronize(); R.barrier()
        e_ms = R.max_over_ranks(e0.elapsed_time(e1), device)
        e2e = {"value": units_all * e_steps / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": e_steps, "ms_per_step": e_ms / e_steps}
        A.asap_check(ctx)
        # both buffer sets carried the same batch: what came back must agree with a directly run step
        A.asap_prune_step(ctx, dev_in[0], params, out, stream)
        torch.cuda.synchronize()
        for j in range(2):
            if not (torch.equal(host_out[j]["keep_idx"], out.keep_idx.cpu()) and
                    torch.equal(host_out[j]["out_hidden"], out.out_hidden[:n_out_rows].cpu())):
                raise RuntimeError("end-to-end leg: the results read back differ from a directly run step")
        del host, host_out, dev_out
    graph = None
    t["graph"] = None
    S.free()

    if rank != 0:
        R.shutdown()
        return

    # ---- roofline: every kernel, and the dominant one on its own key
    alg = algorithmic(batch, keep_k, rank_visual)
    kernels = kernel_table(ktimes, alg, peaks, peak_kind, {} if rank_visual else load_traffic(args.workload))
    roofline = dominant_roofline(kernels)

    # ---- the other configurations, briefly, and the progressive schedule
    others = None
    if solo and not args.no_others:
        others = {}
        for name in ("c1", "c2", "c3"):
            if name == args.workload:
                continue
            b2 = W.config(name)
            rec, S2 = short_run(A, name, b2, b2.keep_k, device, local, stream, peaks, peak_kind, args.other_steps)
            S2.free()
            if name == "c1":      # the latency case also with its 22 MB of inputs resident in L2
                warm, S3 = short_run(A, name, b2, b2.keep_k, device, local, stream, peaks, peak_kind, args.other_steps,
                                     n_copies=1)
                S3.free()
                rec["latency_us_rotated_inputs"] = rec["ms_per_step"] * 1e3
                rec["latency_us_l2_warm"] = warm["ms_per_step"] * 1e3
                rec["l2_warm_kernel_us"] = warm["kernel_us"]
            others[name] = rec
        others["c5_schedule"] = c5_schedule(A, device, local, stream, peaks, peak_kind, args.other_steps)

    # ---- CPU oracle baseline on a bounded sample
    cpu = None
    if solo and not args.no_cpu_baseline:
        v, secs, done, threads = time_oracle(batch, keep_k, budget_s=args.cpu_budget)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{done} sequence evaluations over the {batch.B} sequences of {args.workload} "
                         f"(batch walked {done / batch.B:.1f} times), {secs:.1f} s, float64 numpy; {CORES_NOTE}"}

    step_s = total_ms_max * 1e-3 / args.steps
    line = {
        "metric": METRIC, "value": units_all / step_s, "unit": UNIT, "n_gpus": size, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {WORKLOADS[args.workload]}" +
                               (f" -- PREFIX of {batch.B} sequences" if args.sequences else ""),
                   "sequences_per_gpu": batch.B,
                   "visual_tokens_per_gpu": units, "keep_k": keep_k, "ranking_rows": "image span + text span" if rank_visual else "text span",
                   "l2": (f"inputs rotate over {n_copies} device copies ({n_copies * S.in_bytes / 2**20:.0f} MiB) "
                          f"so no step finds its inputs in the {L2_BYTES // 2**20} MiB L2"),
                   "timed_as": t["timed_as"],
                   "parallelism": "replicas only (one batch per GPU, no collective)"},
        "latency_us": {"p10": per_step[len(per_step) // 10] * 1e3, "p50": per_step[len(per_step) // 2] * 1e3,
                       "p90": per_step[(len(per_step) * 9) // 10] * 1e3, "samples": len(per_step)},
        "clocks": clocks, "e2e": e2e, "gpu_launches": t["launches"], "roofline": roofline, "kernels": kernels,
        "sustained": sustained, "other_workloads": others,
        "cpu_baseline": cpu, "kv_compaction": kv, "staged_entry_points": staged, "consolidate_within_kept": cons, "masked_attention": attn, "direct_launch": direct,
    }
    print(json.dumps(line))
    R.shutdown()


# ------------------------------------------------------------------------------------------
# launching the ranks ourselves
# ------------------------------------------------------------------------------------------
def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(n, argv):
    """`--gpus N` without a launcher: start the N ranks as children of this process, one per GPU, with the
    environment a launcher would give them (rendezvous on 127.0.0.1); rank 0's line is this process's
    output.  Returns the largest exit code."""
    port = free_port()
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + argv, env=env))
    codes = [p.wait() for p in procs]
    return max(abs(c) for c in codes)


def run_rendezvous_check(args):
    """Host-only check of the multi-rank plumbing (no GPU, gloo): every rank joins, meets the others at a
    barrier and takes part in the two reductions the benchmark uses; rank 0 prints what it saw."""
    rank, size, local = R.init("gloo")
    R.barrier()
    slowest = R.max_over_ranks(1.0 + rank)
    total = R.sum_over_ranks(100.0)
    R.barrier()
    if rank == 0:
        print(json.dumps({"impl": "rendezvous-check", "n_gpus": size, "slowest": slowest, "total": total}))
    R.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default 200 for the CUDA arm, 20 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference", "rendezvous-check"])
    ap.add_argument("--workload", default="c4", choices=sorted(WORKLOADS))
    ap.add_argument("--rank-rows", default="text", choices=["text", "visual+text"],
                    help="query rows whose Eq. 4 probabilities rank the visual keys (default: the text span)")
    ap.add_argument("--sequences", type=int, default=None,
                    help="only the first N sequences of the workload (profiling captures; the line's config says so)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=12, help="timed end-to-end steps (at most --steps)")
    ap.add_argument("--kv-layers", type=int, default=3,
                    help="also time KV-cache compaction of this many layers (0 = skip)")
    ap.add_argument("--consolidate-threshold", type=float, default=0.8,
                    help="also time asap_consolidate (Sec. 4.2 inside the kept set) with this threshold t")
    ap.add_argument("--no-graph", action="store_true", help="time directly launched steps instead of graph replays")
    ap.add_argument("--direct-steps", type=int, default=50,
                    help="also time this many directly launched steps when the headline is a graph replay (0 = skip)")
    ap.add_argument("--staged-iters", type=int, default=5,
                    help="also call asap_score / asap_select / asap_merge one by one this many times (0 = skip)")
    ap.add_argument("--consolidate-iters", type=int, default=20, help="timed asap_consolidate calls (0 = skip)")
    ap.add_argument("--attention-iters", type=int, default=5,
                    help="also time asap_attention (the layer's attention under the SG-BiMask) this many times (0 = skip)")
    ap.add_argument("--sustained-s", type=float, default=1.2,
                    help="seconds of back-to-back steps for the sustained leg (0 = skip)")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--other-steps", type=int, default=60, help="timed steps of each of the other configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--ref-sequences", type=int, default=1,
                    help="--impl reference: sequences of the workload the oracle prunes per step")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.steps is None:
        args.steps = 200 if args.impl == "cuda" else 20
    if args.impl == "reference":
        run_reference(args)
    elif args.impl == "rendezvous-check":
        run_rendezvous_check(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
