"""Benchmark of the ASAP prune step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1..c6] [--impl reference]

A step is one pass of the whole prune step (attention mass, salience, mask, masked ranking
scores, top-k, cosine assignment, weighted merge, compaction) over one synthetic batch.  The
default workload is the LLaVA-1.5-7B-shaped batch of 16 sequences (576 visual tokens, ragged
text, keep 64).  One JSON line is printed by rank 0:

  value          visual tokens per second, inputs resident in HBM, all ranks together; the timed steps
                 are replayed from a CUDA graph holding one step per device copy of the inputs
                 (config.timed_as; --no-graph times directly launched steps, which the line also
                 reports as direct_launch)
  e2e            the same with inputs in pinned host memory: every step copies them to the
                 device, runs the step through the C ABI and reads the shortened batch back (the
                 copies of neighbouring steps overlap: two sets of buffers, three streams)
  roofline       the kernel with the largest share of the step, against the measured peak
  kernels        per-kernel device time (CUDA events recorded by the library on its stream)
  cpu_baseline   the float64 CPU oracle timed on this host's cores on a few sequences

With --impl reference the CPU oracle alone is timed (rank 0 only).
With N > 1 every rank prunes its own batch of the same shape (sequences are independent, there
is no exchange step): the ranks only meet at the barriers around the timed region.
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
    "c4": "LLaVA-NeXT AnyRes batch 64: 35 system + 2880 visual + text U[32,256], D=4096, 32x128 heads, keep 576",
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


# ------------------------------------------------------------------------------------------
# algorithmic traffic / work of each kernel for one launch over the whole batch
# ------------------------------------------------------------------------------------------
def algorithmic(batch, keep_k, rank_visual=False):
    """Bytes each kernel must move and flops it must do, from the problem sizes alone:
    every operand it consumes read once, every result written once (bf16 = 2 bytes)."""
    D = batch.D
    out = {name: {"bytes": 0, "flops": 0} for name in
           ("qsum", "mass_salience", "score", "head_sum", "select", "kept_gather", "sim", "merge_compact",
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
def time_oracle(batch, keep_k, budget_s=12.0, max_samples=None):
    """Runs the float64 oracle sequence by sequence until `budget_s` of CPU time is used or the
    batch is exhausted; returns (visual tokens per second, seconds, sequences, threads)."""
    from oracle import asap_oracle as O
    import numpy as np

    def bits(t):   # bf16 tensor -> uint16 bit patterns, the form the oracle takes
        return t.contiguous().view(torch.int16).numpy().view(np.uint16)
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
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
    sample = f"{batch.B} sequence(s) of {args.workload} per step, float64 numpy oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": f"{args.workload}: {WORKLOADS[args.workload]}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------
def device_copies(A, batch, device, n_copies):
    first = A.make_inputs(batch, device)
    copies = [first]
    import dataclasses
    for _ in range(n_copies - 1):
        copies.append(dataclasses.replace(first, q=first.q.clone(), k=first.k.clone(),
                                          hidden=first.hidden.clone(), pos_ids=first.pos_ids.clone()))
    return copies


def run_cuda(args):
    from paper_2603_14549_b200 import binding as A   # raises if libasap.so is missing: no fallback
    rank, size, local = R.init("nccl")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (B200); there is no CPU path")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    peaks, peak_kind = load_peaks()

    seed = R.replica_seed(W.BASE_SEED + int(args.workload[1]) - 1, rank)
    batch = W.config(args.workload, seed=seed)
    keep_k = batch.keep_k
    params = A.Params(keep_k=keep_k)
    units = int(batch.vis_len.sum())
    in_bytes = sum(t.numel() * t.element_size() for t in (batch.q, batch.k, batch.hidden, batch.pos_ids))
    n_copies = max(2, min(64, -(-(8 * L2_BYTES) // in_bytes)))
    ctx = A.asap_init(local, max_total_tokens=batch.total, max_B=batch.B, max_H=batch.H, max_D=batch.D,
                      max_keep_rows=batch.B * keep_k)
    copies = device_copies(A, batch, device, n_copies)
    out = A.alloc_outputs(copies[0], keep_k)
    stream = torch.cuda.Stream(device=device)     # a stream of our own: the legacy stream cannot be captured
    torch.cuda.set_stream(stream)

    rank_visual = args.rank_rows == "visual+text"
    if rank_visual:       # Eq. 3 acts on these rows; the score kernel becomes a dense, tensor-pipe-heavy pass
        import dataclasses
        rs = batch.vis_start.to(device)
        rl = (batch.vis_len + batch.text_len).to(device)
        copies = [dataclasses.replace(c, rank_start=rs, rank_len=rl, max_rank=int((batch.vis_len + batch.text_len).max()))
                  for c in copies]

    def step(i):
        A.asap_prune_step(ctx, copies[i % n_copies], params, out, stream)

    # ---- device-resident timing
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    A.asap_check(ctx)
    # The timed steps are replayed from a CUDA graph that holds one step per device copy of the inputs
    # (the library's calls are capturable: no allocation, no synchronisation, the side stream joins back
    # inside the call), K / copies replays = exactly K steps.  --no-graph, or a K that the number of
    # copies does not divide, times directly launched steps instead.
    graph, per_replay = None, 1
    if not args.no_graph and args.steps % n_copies == 0:
        try:
            c0 = A.asap_launch_count(ctx)
            graph = torch.cuda.CUDAGraph()
            graph.capture_begin()
            for i in range(n_copies):
                step(i)
            graph.capture_end()
            launches_per_replay = A.asap_launch_count(ctx) - c0
            graph.replay()
            torch.cuda.synchronize()
            A.asap_check(ctx)
            per_replay = n_copies
        except Exception as ex:                      # capture not available: fall back to direct launches
            print(f"bench.py: graph capture failed ({ex!r}); timing directly launched steps", file=sys.stderr)
            graph, per_replay = None, 1
    n_marks = args.steps // per_replay
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_marks + 1)]
    launches0 = A.asap_launch_count(ctx)
    R.barrier(); torch.cuda.synchronize()
    wall_begin = time.time()
    marks[0].record(stream)
    for i in range(n_marks):
        if graph is not None:
            graph.replay()
        else:
            step(args.warmup + i)
        marks[i + 1].record(stream)
    torch.cuda.synchronize(); R.barrier()
    wall_end = time.time()
    clocks = sampler.stop(wall_begin, wall_end) if rank == 0 else None
    launches = launches_per_replay * n_marks if graph is not None else A.asap_launch_count(ctx) - launches0
    total_ms = marks[0].elapsed_time(marks[-1])
    per_step = sorted(marks[i].elapsed_time(marks[i + 1]) / per_replay for i in range(n_marks))
    A.asap_check(ctx)
    timed_as = (f"CUDA graph of {n_copies} steps (one per input copy) replayed {n_marks} times" if graph is not None
                else "directly launched steps")
    total_ms_max = R.max_over_ranks(total_ms, device)
    units_all = R.sum_over_ranks(units, device)

    # ---- per-kernel device times: the same steps again with the library's own events on
    A.asap_profile(ctx, True)
    for i in range(min(args.steps, 1000)):        # the library times at most 16384 events between reads
        step(args.warmup + i)
    torch.cuda.synchronize()
    ktimes = A.asap_profile_read(ctx)
    A.asap_profile(ctx, False)

    # ---- the same steps launched directly through the API, reported beside the headline
    direct = None
    if graph is not None and args.direct_steps > 0:
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(3):
            step(i)
        torch.cuda.synchronize()
        d0.record(stream)
        for i in range(args.direct_steps):
            step(i)
        d1.record(stream)
        torch.cuda.synchronize()
        direct = {"us_per_step": d0.elapsed_time(d1) / args.direct_steps * 1e3, "steps": args.direct_steps}

    # ---- KV-cache compaction of the layers up to the pruning layer (next-row feature, timed apart
    # from the step: keys and values of `kv_layers` layers gathered with the step's row map)
    kv = None
    if args.kv_layers > 0:
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
        kv = {"layers": args.kv_layers, "tensors": n_t, "rows_out": n_out, "bytes": kv_bytes, "us": kv_us,
              "GBs": kv_bytes / kv_us / 1e3, "frac_of_hbm_peak": kv_bytes / kv_us / 1e3 / peaks["hbm_gbs"]}
        del kv_src, kv_dst

    # ---- stage 2 as Sec. 4.2 words it (routing inside the kept set, refill by attention mass), timed
    # apart from the step on the step's own stage-1 results
    cons = None
    if args.consolidate_iters > 0 and keep_k < int(batch.vis_len.max()):
        import dataclasses
        p2 = dataclasses.replace(params, sim_threshold=args.consolidate_threshold)
        st1 = [t.clone() for t in (out.mass, out.salience, out.keep_idx, out.drop_idx)]
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
    if args.attention_iters > 0:
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
        h2d = sum(t.numel() * t.element_size() for t in host.values())
        d2h = sum(t.numel() * t.element_size() for t in host_out[0].values())
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
                    for name, t in host.items():
                        getattr(dev_in[j], name).copy_(t, non_blocking=True)
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

        e_steps = max(4, min(args.steps, 30))
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
    A.asap_free(ctx)

    if rank != 0:
        R.shutdown()
        return

    # ---- roofline of the dominant kernel
    alg = algorithmic(batch, keep_k, rank_visual)
    ksum = sum(ms for _, ms in ktimes.values()) or 1.0
    kernels = {}
    for name, (n, ms) in sorted(ktimes.items(), key=lambda kv: -kv[1][1]):
        avg_s = ms / max(n, 1) * 1e-3
        a = alg.get(name, {"bytes": 0, "flops": 0})
        kernels[name] = {"launches": n, "avg_us": avg_s * 1e6, "share": ms / ksum,
                         "alg_GBs": a["bytes"] / avg_s / 1e9 if avg_s > 0 else None,
                         "alg_TFLOPs": a["flops"] / avg_s / 1e12 if avg_s > 0 else None}
    top = next(iter(kernels)) if kernels else None
    roofline = None
    if top:
        a, kt = alg[top], kernels[top]
        hbm_frac = kt["alg_GBs"] / peaks["hbm_gbs"]
        tc_frac = kt["alg_TFLOPs"] / peaks["bf16_tflops"]
        if top in ("sim", "score") and tc_frac > hbm_frac:
            roofline = {"kernel": top, "bound": "tensor", "achieved": kt["alg_TFLOPs"], "peak": peaks["bf16_tflops"],
                        "unit": "TFLOP/s", "frac": tc_frac, "traffic": None, "peak_kind": peak_kind + " (burst)"}
        else:
            roofline = {"kernel": top, "bound": "hbm", "achieved": kt["alg_GBs"], "peak": peaks["hbm_gbs"],
                        "unit": "GB/s", "frac": hbm_frac, "traffic": None, "peak_kind": peak_kind}
        roofline["algorithmic_bytes_per_launch"] = a["bytes"]
        roofline["algorithmic_flops_per_launch"] = a["flops"]
        roofline["avg_launch_us"] = kt["avg_us"]
        traffic_path = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(traffic_path) and not rank_visual:   # DRAM bytes per launch from the committed ncu capture
            with open(traffic_path) as f:
                tr = json.load(f).get(args.workload, {}).get(top)
            roofline["traffic"] = tr

    # ---- CPU oracle baseline on a bounded sample
    cpu = None
    if not args.no_cpu_baseline:
        v, secs, done, threads = time_oracle(batch, keep_k, budget_s=args.cpu_budget)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{done} sequence evaluations over the {batch.B} sequences of {args.workload} "
                         f"(batch walked {done / batch.B:.1f} times), {secs:.1f} s, float64 numpy"}

    step_s = total_ms_max * 1e-3 / args.steps
    line = {
        "metric": METRIC, "value": units_all / step_s, "unit": UNIT, "n_gpus": size, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {WORKLOADS[args.workload]}", "sequences_per_gpu": batch.B,
                   "visual_tokens_per_gpu": units, "keep_k": keep_k, "ranking_rows": "image span + text span" if rank_visual else "text span",
                   "l2": f"inputs rotate over {n_copies} device copies ({n_copies * in_bytes / 2**20:.0f} MiB) "
                         f"so no step finds its inputs in the {L2_BYTES // 2**20} MiB L2",
                   "timed_as": timed_as,
                   "parallelism": "replicas only (one batch per GPU, no collective)"},
        "latency_us": {"p10": per_step[len(per_step) // 10] * 1e3, "p50": per_step[len(per_step) // 2] * 1e3,
                       "p90": per_step[(len(per_step) * 9) // 10] * 1e3},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "kernels": kernels,
        "cpu_baseline": cpu, "kv_compaction": kv, "consolidate_within_kept": cons, "masked_attention": attn, "direct_launch": direct,
    }
    print(json.dumps(line))
    R.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default 2000 for the CUDA arm, 20 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS))
    ap.add_argument("--rank-rows", default="text", choices=["text", "visual+text"],
                    help="query rows whose Eq. 4 probabilities rank the visual keys (default: the text span)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--kv-layers", type=int, default=3,
                    help="also time KV-cache compaction of this many layers (0 = skip)")
    ap.add_argument("--consolidate-threshold", type=float, default=0.8,
                    help="also time asap_consolidate (Sec. 4.2 inside the kept set) with this threshold t")
    ap.add_argument("--no-graph", action="store_true", help="time directly launched steps instead of graph replays")
    ap.add_argument("--direct-steps", type=int, default=500,
                    help="also time this many directly launched steps when the headline is a graph replay (0 = skip)")
    ap.add_argument("--consolidate-iters", type=int, default=50, help="timed asap_consolidate calls (0 = skip)")
    ap.add_argument("--attention-iters", type=int, default=10,
                    help="also time asap_attention (the layer's attention under the SG-BiMask) this many times (0 = skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--ref-sequences", type=int, default=2,
                    help="--impl reference: sequences of the workload the oracle prunes per step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.steps is None:
        args.steps = 2000 if args.impl == "cuda" else 20
    if args.impl == "reference" and args.steps > 100:
        args.ref_sequences = 1          # many steps: the smallest sample, one sequence per step
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
