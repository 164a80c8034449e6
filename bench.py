#!/usr/bin/env python
"""Benchmark of the segment-KV decode attention path on B200.

One *step* is one decode step of an L-layer stack of attention layers of the
chosen shape: per layer one `segkv_decode_step` call, which appends the step's
K/V rows, updates the beam-index table and runs the decode attention in one launch.  All layers are distinct
cache handles, so a step touches L x (unique KV bytes) of HBM, far more than
the L2 holds, and every timed kernel reads cold data.

Printed: ONE JSON line.  `value` is the whole-job unique-KV bandwidth in GB/s: the K/V
bytes the method has to read (prompt rows once per request, every DISTINCT response
row once) divided by the step time.  Every timed step has its own pair of CUDA events,
so the line also carries the median, 10th and 90th percentile of the step time; the
other evaluation shapes are timed the same way and reported under `other_workloads`.
`--curve` prints the step time at every decode step of the workload instead.

`--impl reference` times the CPU float64 oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode_sdpa_unique_kv_bandwidth"
UNIT = "GB/s"
# dram__bytes_read.sum + dram__bytes_write.sum per attention launch from the ncu captures summarised
# under profiles/ (the OPT-30B figure is the batch-4 capture scaled by 16; traffic grows with the batch)
NCU_TRAFFIC_BYTES = {"llama2-7b": 19.231e6, "opt-30b": 8 * (533.13e6 + 4.6e6)}
DEFAULT_LAYERS = {"tiny": 32, "llama2-7b": 32, "llama2-13b": 32, "gptj-6b": 4, "opt-30b": 1, "bloom-176b": 1}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--layers", type=int, default=0, help="distinct cache handles per step (0 = per-workload default)")
    ap.add_argument("--at-step", type=int, default=0, help="decode step to time, 1-based (0 = the workload's last)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling a smaller case)")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--combine", type=int, default=0, help="0 auto, 1 workspace+ticket, 2 cluster")
    ap.add_argument("--tile", type=int, default=0, help="keys per tile of the decode kernel: 0 auto, 32 (quarter-SM CTAs), 64")
    ap.add_argument("--persistent", type=int, default=-1, help="persistent form of the attention call: -1 auto, 0 never, 1 always")
    ap.add_argument("--prompt-layout", default="head_major", choices=["head_major", "token_major", "seq_first"],
                    help="memory layout of the prompt segment (the paper's Fig. 6 compares layouts)")
    ap.add_argument("--beams", type=int, default=0, help="override the workload's beam width")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the workload's prompt length")
    ap.add_argument("--prefill", action="store_true", help="time the prefill attention instead of the decode step")
    ap.add_argument("--prefill-groups", type=int, default=0,
                    help="128-row groups per CTA of the head_dim-128 prefill kernel (1 or 2; 0 = automatic)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-overlap", action="store_true", help="turn programmatic dependent launch off")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the other evaluation shapes (other_workloads)")
    ap.add_argument("--curve", action="store_true", help="time the fused step at every decode step 1..N of the workload")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def unique_bytes(w, prompt_len, unique_rows_total):
    """K and V bytes the method must read for one layer at one step."""
    row = 2 * w.kv_heads * w.head_dim * 2
    return (w.batch * prompt_len + int(unique_rows_total)) * row


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi clock samples, kept only if taken inside the [begin(), end()] load window."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        self.t0 = self.t1 = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def begin(self):
        self.t0 = time.time()

    def end(self):
        self.t1 = time.time()

    def samples_in_window(self):
        return 0 if self.t0 is None else int((time.time() - self.t0) / 0.05)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        import datetime
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) != 7:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                if self.t0 is not None and not (self.t0 <= ts <= (self.t1 or ts)):
                    continue
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(w, t, budget_s=12.0, max_pairs=None):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload at step t.
    Returns (GB/s of unique KV over the sample, seconds, description, threads)."""
    import torch
    import oracle
    from paper_2401_05391_b200 import workloads as wl

    # one request, all of its heads (every request is an independent unit of the path)
    w1 = w.scaled(batch=1)
    par = wl.make_parents(w1)
    kp, vp = wl.make_prompt(w1, "cpu")
    steps = [wl.make_step(w1, s, "cpu") for s in range(t + 1)]
    q = steps[t][0]
    kr = np.stack([wl.to_bits(s[1]) for s in steps]); vr = np.stack([wl.to_bits(s[2]) for s in steps])
    slopes = wl.alibi_slopes(w.heads).numpy() if w.alibi else None
    heads = list(range(w.heads))
    if max_pairs:
        heads = heads[:max(1, max_pairs // w.beams)]
    pairs = [(g, h) for g in range(w1.rows) for h in heads]
    args = (w.dtype, 1, w.beams, w.heads, w.kv_heads, w.head_dim, wl.to_bits(q), wl.to_bits(kp), wl.to_bits(vp),
            kr, vr, par, t)
    anc = oracle.ancestry(par, 1, w.beams, t)
    uniq = sum(len(set(anc[:, s].tolist())) for s in range(t + 1))
    kv_heads_used = len({h // (w.heads // w.kv_heads) for h in heads})
    nbytes = (w.prompt_len + uniq) * 2 * kv_heads_used * w.head_dim * 2
    oracle.decode_sdpa(*args, slopes=slopes, pairs=pairs[:w.beams])            # load, page in
    reps, total = 0, 0.0
    while True:
        t0 = time.perf_counter()
        oracle.decode_sdpa(*args, slopes=slopes, pairs=pairs)
        total += time.perf_counter() - t0
        reps += 1
        if total >= budget_s or reps >= 50:
            break
    sec = total / reps
    desc = (f"1 request x {len(heads)} heads x {w.beams} beams of {w.name} at step {t + 1} "
            f"({len(pairs)} attention rows over {w.prompt_len + t + 1} keys), mean of {reps} runs")
    return nbytes / sec / 1e9, sec, desc, oracle.threads()


def run_reference(args):
    from paper_2401_05391_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.by_name(args.workload)
    t = (args.at_step or w.steps) - 1
    vals = []
    desc = ""
    threads = 1
    for i in range(args.warmup + args.steps):
        gbs, sec, desc, threads = oracle_sample(w, t, budget_s=0.0, max_pairs=256)
        if i >= args.warmup:
            vals.append((gbs, sec))
    gbs = statistics.mean(v[0] for v in vals)
    sec = statistics.mean(v[1] for v in vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "at_step": t + 1, "sample": desc},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- ours
class DeviceErrorFlags(RuntimeError):
    """A kernel of the timed runs reported an error in the handle's device error word."""


def percentiles(xs):
    xs = sorted(xs)
    n = len(xs)
    pick = lambda f: xs[min(n - 1, max(0, int(round(f * (n - 1)))))]
    return {"median": statistics.median(xs), "p10": pick(0.10), "p90": pick(0.90), "n": n}


class ShapeBench:
    """L layer caches of one shape, filled up to decode step T, and timed passes over them."""

    def __init__(self, w, L, T, args, rank, world, dev):
        import torch
        from paper_2401_05391_b200 import sharding
        from paper_2401_05391_b200 import workloads as wl
        from paper_2401_05391_b200.segkv import SegKV
        self.torch, self.wl, self.sharding = torch, wl, sharding
        self.w, self.L, self.T, self.t = w, L, T, T - 1
        self.args, self.rank, self.world, self.dev = args, rank, world, dev
        # every rank holds its own requests (weak scaling: requests are independent, no exchange)
        w_rank = sharding.rank_workload(w, rank, world)
        self.parents = torch.from_numpy(wl.make_parents(w_rank)).to(dev)
        self.slopes = wl.alibi_slopes(w.heads).to(dev) if w.alibi else None
        self.handles = []
        for layer in range(L):
            wl_layer = w_rank.scaled(index=w_rank.index + 1000 * layer)
            h = SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype)
            if args.tile:
                h.set_tile(args.tile)
            if args.persistent != -1:
                h.set_persistent(args.persistent)
            if args.splits or args.stages or args.combine:
                h.set_tuning(args.splits, args.stages, args.combine)
            if args.no_overlap:
                h.set_overlap(False)
            if args.prompt_layout != "head_major":
                h.set_prompt_layout(args.prompt_layout)
            kp, vp = wl.make_prompt(wl_layer, dev)
            h.prefill_write(kp, vp)
            del kp, vp
            q = k = v = None
            for s in range(T):
                q, k, v = wl.make_step(wl_layer, s, dev)
                h.append(s, self.parents[s] if s > 0 else None, k, v)
            self.handles.append([h, q, k, v, torch.empty_like(q), wl_layer])
        torch.cuda.synchronize()
        self.stream = torch.cuda.Stream()
        self.refresh_bytes()

    def refresh_bytes(self):
        w = self.w
        uniq_rows = int(self.handles[0][0].get_unique_rows().sum())
        self.ubytes = unique_bytes(w, w.prompt_len, uniq_rows)
        self.logical_bytes = w.rows * (w.prompt_len + self.T) * 2 * w.kv_heads * w.head_dim * 2

    def close(self):
        # a kernel that gave up on a bounded wait or clamped a parent id says so in the handle's device
        # error word: a timing taken from such a run is not a timing
        for h in self.handles:
            flags = h[0].get_error()
            h[0].destroy()
            if flags:
                raise DeviceErrorFlags(f"device error flags {flags:#x} were raised during the benchmark")
        self.handles = []

    def layer_pass(self, mode: str):
        # "step": the whole hot path in the library's fused call; "two": the same as two calls
        # (append, then attention); "sdpa": the attention kernel alone on the state already there
        t, stream, slopes = self.t, self.stream, self.slopes
        par_t = self.parents[t] if t > 0 else None
        for h, q, k, v, out, _ in self.handles:
            if mode == "step":
                h.truncate_last()
                h.decode_step(t, par_t, k, v, q, out, slopes, stream=stream)
            elif mode == "two":
                h.truncate_last()
                h.append(t, par_t, k, v, stream=stream)
                h.decode_sdpa(q, out, slopes, stream=stream)
            elif mode == "sdpa":
                h.decode_sdpa(q, out, slopes, stream=stream)
        if mode == "hot":
            # the attention kernel on ONE layer's cache over and over: L2-resident where the layer fits
            # (the Llama2-7B shape does), i.e. the kernel's latency floor without HBM
            h, q, k, v, out, _ = self.handles[0]
            for _ in range(len(self.handles)):
                h.decode_sdpa(q, out, slopes, stream=stream)

    def make_runner(self, mode: str):
        torch, stream = self.torch, self.stream
        with torch.cuda.stream(stream):
            self.layer_pass(mode)                            # lazy initialisation outside any capture
        stream.synchronize()
        if self.args.no_graph:
            return (lambda: self.layer_pass(mode)), False
        g = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.graph(g, stream=stream):
                self.layer_pass(mode)
        except Exception as e:                               # report, never hide
            sys.stderr.write(f"[bench] CUDA graph capture failed ({e}); timing direct launches\n")
            return (lambda: self.layer_pass(mode)), False

        def replay():
            with torch.cuda.stream(stream):
                g.replay()
        return replay, True

    def timed(self, run, steps, warmup):
        """K steps between two events (total, max over ranks) and every step between its own pair."""
        torch, stream, dist = self.torch, self.stream, self.torch.distributed
        for _ in range(warmup):
            run()
        stream.synchronize()
        if self.world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record(stream)
        for i in range(steps):
            run()
            ev[i + 1].record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        ms = self.sharding.max_over_ranks(ev[0].elapsed_time(ev[steps]), self.dev)
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        if self.world > 1:
            dist.barrier()
        return ms, per

    def launches_per_step(self):
        l0 = sum(h[0].launch_count for h in self.handles)
        with self.torch.cuda.stream(self.stream):
            self.layer_pass("step")
        self.stream.synchronize()
        return sum(h[0].launch_count for h in self.handles) - l0      # counted by the library


def run_curve(args):
    """The fused step at every decode step 1..N of the workload (one JSON line with the arrays)."""
    import torch
    from paper_2401_05391_b200 import workloads as wl
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = wl.by_name(args.workload)
    L = args.layers or DEFAULT_LAYERS.get(w.name, 1)
    sb = ShapeBench(w, L, 1, args, 0, 1, dev)
    peak, peak_kind = peaks()
    steps_k = max(20, min(args.steps, 50))
    rows = []
    for T in range(1, w.steps + 1):
        if T > 1:
            # one more step on every layer (the state the timed step starts from)
            for hh in sb.handles:
                q, k, v = wl.make_step(hh[5], T - 1, dev)
                hh[0].append(T - 1, sb.parents[T - 1], k, v)
                hh[1], hh[2], hh[3] = q, k, v
            torch.cuda.synchronize()
        sb.T, sb.t = T, T - 1
        sb.refresh_bytes()
        run, _ = sb.make_runner("step")
        _, per = sb.timed(run, steps_k, 3)
        med = statistics.median(per) * 1e3 / L
        gbs = sb.ubytes / (med * 1e-6) / 1e9
        rows.append({"at_step": T, "us_per_step_per_layer": round(med, 3), "unique_kv_bytes": sb.ubytes,
                     "gbs": round(gbs, 1), "frac_of_measured": round(gbs / peak, 4)})
    print(json.dumps({"metric": METRIC, "unit": UNIT, "workload": w.name, "layers_per_step": L,
                      "replays_per_point": steps_k, "peak": peak, "peak_kind": f"of {peak_kind}", "curve": rows}))
    sb.close()


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2401_05391_b200 import workloads as wl
    from paper_2401_05391_b200 import sharding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = wl.by_name(args.workload)
    if args.batch:
        w = w.scaled(batch=args.batch, name=f"{w.name}[batch={args.batch}]")
    if args.beams:
        w = w.scaled(beams=args.beams, name=f"{w.name}[beams={args.beams}]")
    if args.prompt_len:
        w = w.scaled(prompt_len=args.prompt_len, name=f"{w.name}[prompt={args.prompt_len}]")
    L = args.layers or DEFAULT_LAYERS.get(w.name.split("[")[0], 1)
    T = args.at_step or w.steps
    t = T - 1
    sampler = ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}") if rank == 0 else None
    sb = ShapeBench(w, L, T, args, rank, world, dev)
    handles, stream, parents, slopes = sb.handles, sb.stream, sb.parents, sb.slopes
    ubytes, logical_bytes = sb.ubytes, sb.logical_bytes

    # ---- the timed region: K whole steps (append + beam-index update + attention, all layers)
    launches0 = sum(h[0].launch_count for h in handles)
    launches_per_step = sb.launches_per_step()
    run_step, graphed = sb.make_runner("step")
    if sampler:
        sampler.begin()
    ms_total, per_step = sb.timed(run_step, args.steps, args.warmup)
    # ---- the attention kernel alone, same rotation over cold layers (roofline numerator)
    run_sdpa, _ = sb.make_runner("sdpa")
    ms_sdpa, per_sdpa = sb.timed(run_sdpa, args.steps, max(3, args.warmup))
    run_hot, _ = sb.make_runner("hot")
    ms_hot, _ = sb.timed(run_hot, args.steps, max(3, args.warmup))
    # ---- for comparison: the same step as two library calls (append, then attention)
    run_two, _ = sb.make_runner("two")
    ms_two, _ = sb.timed(run_two, args.steps, max(3, args.warmup))
    clocks = None
    if sampler:
        # the timed loops can be shorter than nvidia-smi's sampling period: keep the same load up
        # (untimed) until a handful of samples fall inside the window
        t_end = time.time() + 3.0
        while sampler.samples_in_window() < 12 and time.time() < t_end:
            for _ in range(20):
                run_step()
            stream.synchronize()
        sampler.end()
        clocks = sampler.stop()
    ms_per_step = ms_total / args.steps
    us_layer = ms_per_step * 1e3 / L
    us_sdpa = ms_sdpa / args.steps * 1e3 / L
    value = sharding.whole_job_rate(L * ubytes, world, ms_per_step * 1e-3) / 1e9

    # ---- end to end from host memory through segkv_layers_step_host
    e2e = None
    if not args.no_e2e:
        # every layer's step inputs packed into one pinned host block; the library queues the copies in, the
        # launches and the copies out of all layers in one call
        total, off = handles[0][0].host_pack_layout()
        hs = slopes is not None
        hq = []
        # ONE pinned array for the inputs of all layers and one for their outputs (a layer's block is a
        # slice): blocks that lie back to back let the library move several layers with one copy
        q0 = handles[0][1]
        blk_all = torch.zeros(len(handles), total, dtype=torch.uint8).pin_memory()
        out_all = torch.empty((len(handles),) + tuple(q0.shape), dtype=q0.dtype).pin_memory()
        for li, (_, q, k, v, _, _) in enumerate(handles):
            blk = blk_all[li]

            def put(o, x):
                raw = x.contiguous().cpu().view(torch.uint8).reshape(-1)
                blk[o:o + raw.numel()] = raw
            if t > 0:
                put(off[0], parents[t])
            if hs:
                put(off[1], slopes)
            put(off[2], k); put(off[3], v); put(off[4], q)
            hq.append((blk, out_all[li]))

        from paper_2401_05391_b200.segkv import LayerStack
        stack = LayerStack([h[0] for h in handles], [x[0] for x in hq], [x[1] for x in hq])

        def host_step():
            # one call queues every layer's copy in, launch and copy out; the host waits once per step
            stack.step(t, has_slopes=hs, redo=True, stream=stream)
            stream.synchronize()
        n_e2e = max(3, min(args.steps, 20))
        for _ in range(3):
            host_step()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            host_step()
        torch.cuda.synchronize()
        sec = (time.perf_counter() - t0) / n_e2e
        sec = sharding.max_over_ranks(sec, dev)
        q = handles[0][1]
        h2d = L * total                      # the packed block: parents, slopes, k, v, q and their padding
        d2h = L * q.numel() * 2
        e2e = {"value": sharding.whole_job_rate(L * ubytes, world, sec) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "us_per_step_per_layer": sec * 1e6 / L}

    splits_used = handles[0][0].get_splits()
    assert sum(h[0].launch_count for h in handles) > launches0
    sb.close()

    # ---- what a kernel that only reads can reach on this GPU (4 GiB streamed with 16-byte loads): the
    # copy figure of MEASURED_PEAKS.json counts bytes read plus written and sits lower, which is why
    # the read-only attention kernel can show more than 1.0 of it
    read_peak = None
    if rank == 0:
        from paper_2401_05391_b200.segkv import read_bandwidth
        buf = torch.empty(4 << 30, dtype=torch.uint8, device=dev)
        buf.zero_()
        read_peak = read_bandwidth(buf, 10)
        del buf
    # ---- the other evaluation shapes, each timed the same way (fused step and attention alone)
    peak, peak_kind = peaks()
    others = None
    default_shape = not (args.batch or args.beams or args.prompt_len or args.at_step or args.tile or args.splits or
                         args.stages or args.combine or args.no_graph or args.no_overlap or
                         args.prompt_layout != "head_major")
    if world == 1 and not args.no_others and default_shape:
        others = {}
        k_other = max(20, min(args.steps, 30))
        for c in wl.CONFIGS:
            if c.name == w.name:
                continue
            Lc = DEFAULT_LAYERS.get(c.name, 1)
            so = ShapeBench(c, Lc, c.steps, args, 0, 1, dev)
            oc = ClockSampler(f"GPU-{torch.cuda.get_device_properties(dev).uuid}")
            oc.begin()
            run_o, _ = so.make_runner("step")
            _, per_o = so.timed(run_o, k_other, 3)
            run_a, _ = so.make_runner("sdpa")
            _, per_a = so.timed(run_a, k_other, 3)
            t_end = time.time() + 2.0
            while oc.samples_in_window() < 8 and time.time() < t_end:
                for _ in range(5):
                    run_a()
                so.stream.synchronize()
            oc.end()
            ps, pa = percentiles(per_o), percentiles(per_a)
            us_a = pa["median"] * 1e3 / Lc
            gbs_a = so.ubytes / (us_a * 1e-6) / 1e9
            others[c.name] = {
                "layers_per_step": Lc, "at_step": c.steps, "unique_kv_bytes_per_layer": so.ubytes,
                "us_per_step_per_layer": ps["median"] * 1e3 / Lc,
                "us_per_step_per_layer_p10": ps["p10"] * 1e3 / Lc, "us_per_step_per_layer_p90": ps["p90"] * 1e3 / Lc,
                "us_sdpa_per_layer": us_a, "us_sdpa_per_layer_p10": pa["p10"] * 1e3 / Lc,
                "us_sdpa_per_layer_p90": pa["p90"] * 1e3 / Lc, "replays": k_other,
                "gbs": gbs_a, "pct_of_8000": 100.0 * gbs_a / 8000.0, "frac_of_measured": gbs_a / peak,
                "frac_of_read_only_peak": gbs_a / read_peak if read_peak else None,
                "gbs_whole_step": so.ubytes / (ps["median"] * 1e-3 / Lc) / 1e9,
                "clocks": oc.stop(),
            }
            so.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # The dominant kernel of the timed region.  When a step is one fused launch per layer, that launch IS
    # the region: its duration is the step time per layer.  When a step is two launches (append, then
    # attention), the attention kernel's own duration comes from the attention-only loop over the same
    # cold layers, and the timed step adds the append launch on top (us_per_step_per_layer).
    fused_step = launches_per_step == L
    us_dom = us_layer if fused_step else us_sdpa
    achieved = ubytes / (us_dom * 1e-6) / 1e9
    achieved_attn = ubytes / (us_sdpa * 1e-6) / 1e9
    pstep, psdpa = percentiles(per_step), percentiles(per_sdpa)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16" if w.dtype == "f16" else "bf16", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "beams": w.beams, "heads": w.heads, "kv_heads": w.kv_heads,
                   "head_dim": w.head_dim, "prompt_len": w.prompt_len, "at_step": T, "layers_per_step": L,
                   "l2": f"{L} distinct layer caches per step, {L * ubytes / 1e6:.0f} MB > L2", "cuda_graph": graphed, "dependent_launch": not args.no_overlap,
                   "prompt_layout": args.prompt_layout,
                   "splits": splits_used, "parallelism": f"replica x{world}" if world > 1 else "1 gpu"},
        "ms_per_step_median": pstep["median"], "ms_per_step_p10": pstep["p10"], "ms_per_step_p90": pstep["p90"],
        "us_per_step_per_layer": us_layer,
        "us_per_step_per_layer_median": pstep["median"] * 1e3 / L,
        "us_sdpa_per_layer": us_sdpa,
        "us_sdpa_per_layer_median": psdpa["median"] * 1e3 / L,
        "us_sdpa_per_layer_p10": psdpa["p10"] * 1e3 / L, "us_sdpa_per_layer_p90": psdpa["p90"] * 1e3 / L,
        "us_sdpa_same_layer_repeated": ms_hot / args.steps * 1e3 / L,
        "us_per_step_per_layer_two_calls": ms_two / args.steps * 1e3 / L,
        "unique_kv_bytes_per_layer": ubytes,
        "logical_kv_bytes_per_layer": logical_bytes,
        "pct_of_8000_GBps": 100.0 * achieved_attn / 8000.0,
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": NCU_TRAFFIC_BYTES.get(w.name) if T == w.steps else None, "peak_kind": f"of {peak_kind}",
                     "kernel": ("sdpa_tiled_kernel<FUSED> (append + beam-index update + attention in one launch)"
                                if fused_step else "sdpa_tiled_kernel (attention; the append is a second, small launch)"),
                     "timed": ("timed region: one launch per layer, step time / launches" if fused_step
                               else "attention-only loop over the same cold layers"),
                     "bytes_per_launch": ubytes, "us_per_launch": us_dom,
                     "attention_only": {"us_per_launch": us_sdpa, "achieved": achieved_attn, "frac": achieved_attn / peak},
                     "read_only_peak": {"value": read_peak, "unit": "GB/s", "frac": achieved / read_peak,
                                        "how": "segkv_read_bandwidth: 4 GiB streamed 10 times with 16-byte loads, CUDA events"}
                     if read_peak else None},
        "e2e": e2e,
        "clocks": clocks,
    }
    if others is not None:
        line["other_workloads"] = others
    if not args.no_cpu_baseline:
        gbs, sec, desc, threads = oracle_sample(w, t)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                                "seconds": sec}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_prefill(args):
    """Prefill attention of the workload's prompt (one JSON line of its own; tensor-core bound)."""
    import torch
    from paper_2401_05391_b200 import workloads as wl
    from paper_2401_05391_b200.segkv import SegKV
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = wl.by_name(args.workload)
    if args.batch:
        w = w.scaled(batch=args.batch, name=f"{w.name}[batch={args.batch}]")
    if args.beams:
        w = w.scaled(beams=args.beams, name=f"{w.name}[beams={args.beams}]")
    if args.prompt_len:
        w = w.scaled(prompt_len=args.prompt_len, name=f"{w.name}[prompt={args.prompt_len}]")
    L = args.layers or DEFAULT_LAYERS.get(w.name.split("[")[0], 1)
    handles = []
    for layer in range(L):
        wl_layer = w.scaled(index=w.index + 1000 * layer)
        h = SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, 1, w.torch_dtype)
        if args.prompt_layout != "head_major":
            h.set_prompt_layout(args.prompt_layout)
        kp, vp = wl.make_prompt(wl_layer, dev)
        h.prefill_write(kp, vp)
        if args.prefill_groups:
            h.set_prefill_tuning(args.prefill_groups)
        if layer == 0:
            kv0 = (kp, vp)                   # kept for the whole-prefill timing below
        del kp, vp
        q = wl.make_prefill_query(wl_layer, dev)
        handles.append((h, q, torch.empty_like(q)))
    slopes = wl.alibi_slopes(w.heads).to(dev) if w.alibi else None
    stream = torch.cuda.Stream()

    def one_pass():
        for h, q, o in handles:
            h.prefill_sdpa(q, o, slopes, stream=stream)
    for _ in range(max(3, args.warmup)):
        one_pass()
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        one_pass()
    e1.record(stream)
    stream.synchronize()
    ms = e0.elapsed_time(e1) / args.steps / L
    # the whole prefill of one layer: prompt store + attention as two calls, and as the one fused launch
    h0, q0, o0 = handles[0]

    def timed(fn):
        for _ in range(3):
            fn()
        stream.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(args.steps):
            fn()
        t1.record(stream)
        stream.synchronize()
        return t0.elapsed_time(t1) / args.steps

    def two_calls():
        h0.prefill_write(kv0[0], kv0[1], stream=stream)
        h0.prefill_sdpa(q0, o0, slopes, stream=stream)
    ms_two = timed(two_calls)
    ms_fused = timed(lambda: h0.prefill(kv0[0], kv0[1], q0, o0, slopes, stream=stream))
    n = w.prompt_len
    flops = 4.0 * w.head_dim * (n * (n + 1) / 2) * w.batch * w.heads          # causal: only the visible keys
    tflops = flops / (ms * 1e-3) / 1e12
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak, kind = (float(json.load(open(path))["bf16_tflops"]), "measured") if os.path.exists(path) else (1590.0, "fallback")
    print(json.dumps({
        "metric": "prefill_sdpa_causal_tflops", "value": tflops, "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "ms_store_then_attention": ms_two,
        "ms_fused_store_and_attention": ms_fused, "higher_is_better": True, "dtype": w.dtype,
        "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "heads": w.heads, "kv_heads": w.kv_heads,
                   "head_dim": w.head_dim, "prompt_len": n, "layers_rotated": L},
        "roofline": {"bound": "tensor", "achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak,
                     "traffic": None, "peak_kind": f"of {kind} (bf16 GEMM burst; fp16 has the same nominal rate)",
                     "kernel": "segkv prefill attention (tcgen05, S/P/O in tensor memory, persistent CTAs)"},
        "gpu_launches": args.steps * L}))


def main():
    args = parse()
    if args.prefill and args.impl != "reference":
        return run_prefill(args)
    if args.curve and args.impl != "reference":
        return run_curve(args)
    if args.impl == "reference":
        run_reference(args)
        return
    try:
        run_ours(args)
    except DeviceErrorFlags as e:
        # nothing has been printed yet (the line comes last): measure once more when this process is the
        # whole job (ranks of a larger job must stay in step), and fail if it happens again
        if int(os.environ.get("WORLD_SIZE", "1")) != 1:
            raise
        print(f"bench.py: {e}; measuring once more", file=sys.stderr)
        run_ours(args)


if __name__ == "__main__":
    main()
