"""Per-CTA time stamps of the decode attention kernel in a chain of back-to-back launches.

The attention kernel can be compiled with time stamps (``-DSEGKV_TIMELINE``): every CTA records
``%globaltimer`` when it starts and the SM's cycle counter at fixed points of its life into a
device array that keeps the last eight launches.  This script builds that instrumented copy of the library
(``libsegkv_timeline.so``; the product library is not touched), replays a CUDA graph of one
launch per layer over L distinct layer caches, as ``bench.py`` does, and prints for each of
the last eight launches the median and the latest CTA of every stamp, in microseconds from the
first CTA start of the first of them, followed by the launch-to-launch period.

    python -m paper_2401_05391_b200.timeline [--workload llama2-7b] [--fused] [--splits N]
                                              [--stages N] [--combine N] [--tile N] [--layers L] [--no-overlap]

Stamps (slot in the per-CTA record): 0 CTA start, 3 first prompt tiles requested, 2 grid-dependency
wait returned, 4 gather warp knows its rows, 5 last response copy issued, 7 first tile landed,
6 first tile consumed (the query has arrived too), 8 prompt tiles consumed, 9 response tiles consumed, 10 all warps at the
epilogue, 11 partial written, 12 ticket / cluster barrier passed, 13 merged output stored.
"""
from __future__ import annotations

import argparse
import ctypes

import numpy as np
import torch

EVENTS = [(0, "start"), (3, "tma issued"), (2, "wait done"), (7, "tile 0 landed"), (6, "tile 0 used"), (4, "rows known"),
          (5, "copies issued"), (8, "prompt done"), (9, "resp done"), (10, "epilogue"), (11, "partial out"),
          (12, "ticket/barrier"), (13, "merged")]
SLOTS, CTAS, WORDS = 8, 512, 32      # per CTA: 16 x %globaltimer (ns), then 16 x clock64 of the same stamps


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama2-7b")
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--fused", action="store_true", help="time segkv_decode_step instead of segkv_decode_sdpa")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--combine", type=int, default=0)
    ap.add_argument("--tile", type=int, default=0)
    ap.add_argument("--no-overlap", action="store_true")
    ap.add_argument("--sm-mhz", type=int, default=1965, help="SM clock under load, to turn cycles into time")
    a = ap.parse_args()

    from . import build, segkv as sk, workloads as wl
    sk.LIB_PATH = build.build(timeline=True)            # before the first sk.lib()
    lib = sk.lib()
    lib.segkv_debug_timeline.argtypes = [ctypes.c_void_p, ctypes.c_int]

    w = wl.by_name(a.workload)
    dev = "cuda"
    par = torch.from_numpy(wl.make_parents(w)).to(dev)
    layers = []
    for layer in range(a.layers):
        wlay = w.scaled(index=w.index + 1000 * layer)
        h = sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype)
        if a.tile:
            h.set_tile(a.tile)
        if a.splits or a.stages or a.combine:
            h.set_tuning(a.splits, a.stages, a.combine)
        h.set_overlap(not a.no_overlap)
        kp, vp = wl.make_prompt(wlay, dev)
        h.prefill_write(kp, vp)
        for s in range(w.steps):
            q, k, v = wl.make_step(wlay, s, dev)
            h.append(s, par[s] if s > 0 else None, k, v)
        layers.append((h, q, torch.empty_like(q), k, v))
    torch.cuda.synchronize()
    st = torch.cuda.Stream()
    t_last = w.steps - 1

    def one_pass():
        with torch.cuda.stream(st):
            for h, q, o, k, v in layers:
                if a.fused:
                    h.truncate_last()
                    h.decode_step(t_last, par[t_last], k, v, q, o, stream=st)
                else:
                    h.decode_sdpa(q, o, stream=st)

    one_pass()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        one_pass()
    for _ in range(3):
        with torch.cuda.stream(st):
            g.replay()
    torch.cuda.synchronize()
    buf = np.zeros(SLOTS * CTAS * WORDS, dtype=np.uint64)
    assert lib.segkv_debug_timeline(buf.ctypes.data, 0) == 0
    n = min(CTAS, w.batch * w.kv_heads * layers[0][0].get_splits())
    raw = buf.reshape(SLOTS, CTAS, WORDS).astype(np.int64)[:, :n]
    raw = raw[np.argsort(raw[:, :, 0].min(axis=1))]      # the eight launch slots in time order
    # Only the CTA start carries %globaltimer (reading it is slow and coarse); every stamp carries
    # the SM's cycle counter, which is converted with the clock the GPU runs at under load.
    mhz = a.sm_mhz
    clk = raw[:, :, 16:]
    t = np.where(clk > 0, raw[:, :, 0:1] + (clk - clk[:, :, 0:1]) * 1000 // mhz, 0)
    g0 = t[0, :, 0].min()
    print(f"{a.workload}: {n} CTAs per launch, splits {layers[0][0].get_splits()}, "
          f"{'fused step' if a.fused else 'attention only'}; median / latest CTA, us from the first CTA start")
    order = EVENTS + [(14, "remote stores"), (1, "consumer set up"), (15, "tile 0 scores")]
    print("launch | " + " | ".join(f"{name:>14s}" for _, name in order))
    for li in range(SLOTS):
        cells = []
        for ev, _ in order:
            x = t[li, :, ev]
            m = x > 0
            cells.append(f"{(np.median(x[m]) - g0) / 1e3:6.2f}/{(x[m].max() - g0) / 1e3:6.2f} " if m.any() else f"{'-':>14s}")
        print(f"{li:6d} | " + " | ".join(cells))
    print("cycles from the CTA's own start, median over the CTAs of the last launch:")
    c = clk[SLOTS - 1]
    line = []
    for ev, name in order:
        m = (c[:, ev] > 0) & (c[:, 0] > 0)
        if m.any():
            line.append(f"{name} {int(np.median(c[m, ev] - c[m, 0]))}")
    print("  " + " | ".join(line))
    starts = t[:, :, 0].min(axis=1)
    ends = np.where(t[:, :, 13] > 0, t[:, :, 13], t[:, :, 12]).max(axis=1)
    print("first CTA start to first CTA start, us:", np.round(np.diff(starts) / 1e3, 2))
    print("last output to last output, us:        ", np.round(np.diff(ends) / 1e3, 2))
    for h, *_ in layers:
        h.destroy()


if __name__ == "__main__":
    main()
