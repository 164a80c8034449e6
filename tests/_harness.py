"""Drives a synthetic workload through the CUDA library and evaluates the same
bits with the CPU oracle.  Test-side glue only."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2401_05391_b200 import workloads as wl
from paper_2401_05391_b200.segkv import SegKV

ATOL, RTOL = 2e-3, 1e-2   # |gpu - ref| <= ATOL + RTOL*|ref|, the path's stated tolerance


class Run:
    def __init__(self, w: wl.Workload, device="cuda", max_steps=None, max_prompt=None, parents=None,
                 splits=0, stages=0, combine=0, chunk_steps=0, prompt_layout=None,
                 prompt_lens=None, tile=0, persistent=-1):
        self.w, self.device = w, device
        self.h = SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim,
                       w.prompt_len if max_prompt is None else max_prompt,
                       w.steps if max_steps is None else max_steps, w.torch_dtype, chunk_steps=chunk_steps)
        if tile:
            self.h.set_tile(tile)
        if persistent != -1:
            self.h.set_persistent(persistent)
        if splits or stages or combine:
            self.h.set_tuning(splits, stages, combine)
        if prompt_layout is not None:
            self.h.set_prompt_layout(prompt_layout)
        self.parents = wl.make_parents(w) if parents is None else np.ascontiguousarray(parents, np.int32)
        self.parents_dev = torch.from_numpy(self.parents).to(device)
        self.slopes = wl.alibi_slopes(w.heads).to(device) if w.alibi else None
        self.kp = self.vp = None
        if w.prompt_len > 0:
            self.kp, self.vp = wl.make_prompt(w, device)
        self.prompt_lens = None if prompt_lens is None else [int(x) for x in prompt_lens]
        if self.prompt_lens is not None:
            # the padding behind each request's own prompt is poison: the library must never let it through
            for b, n in enumerate(self.prompt_lens):
                self.kp[b, n:] = float("nan")
                self.vp[b, n:] = float("inf")
            self.h.prefill_write_ragged(self.kp, self.vp, self.prompt_lens)
        else:
            self.h.prefill_write(self.kp, self.vp)
        self.k_steps, self.v_steps, self.q_steps = [], [], []

    def close(self):
        self.h.destroy()

    def append_next(self):
        t = self.h.steps
        q, k, v = wl.make_step(self.w, t, self.device)
        self.h.append(t, self.parents_dev[t] if t > 0 else None, k, v)
        self.k_steps.append(k); self.v_steps.append(v); self.q_steps.append(q)
        return t

    def append_next_rope(self, cos, sin, style):
        """Append the next step through segkv_append_rope; the oracle side gets K rows rotated by the
        oracle's own rotary embedding (position = the request's prompt length + step)."""
        w, t = self.w, self.h.steps
        q, k, v = wl.make_step(w, t, self.device)
        self.h.append_rope(t, self.parents_dev[t] if t > 0 else None, k, v, cos, sin, style)
        plens = self.prompt_lens if self.prompt_lens is not None else [w.prompt_len] * w.batch
        pos = np.repeat(np.asarray(plens, np.int64) + t, w.beams * w.kv_heads)          # one per (row, kv head)
        rot = oracle.rope(w.dtype, wl.to_bits(k).reshape(-1, w.head_dim), cos.cpu().numpy()[pos],
                          sin.cpu().numpy()[pos], style)
        k_rot = torch.from_numpy(rot.view(np.int16).reshape(tuple(k.shape))).view(w.torch_dtype).to(self.device)
        self.k_steps.append(k_rot); self.v_steps.append(v); self.q_steps.append(q)
        return t

    def step_fused(self):
        """Append the next step and attend in one fused launch; returns (t, out, q)."""
        t = self.h.steps
        q, k, v = wl.make_step(self.w, t, self.device)
        out = torch.full((self.w.rows, self.w.heads, self.w.head_dim), float("nan"),
                         dtype=self.w.torch_dtype, device=self.device)
        self.h.decode_step(t, self.parents_dev[t] if t > 0 else None, k, v, q, out, self.slopes)
        torch.cuda.synchronize()
        self.k_steps.append(k); self.v_steps.append(v); self.q_steps.append(q)
        return t, out, q

    def advance_to(self, t: int):
        while self.h.steps <= t:
            self.append_next()

    def decode(self, q=None):
        if q is None:
            q = self.q_steps[-1] if self.q_steps else wl.make_step(self.w, 0, self.device)[0]
        out = torch.full((self.w.rows, self.w.heads, self.w.head_dim), float("nan"),
                         dtype=self.w.torch_dtype, device=self.device)
        self.h.decode_sdpa(q, out, self.slopes)
        torch.cuda.synchronize()
        return out, q

    # ------------------------------------------------------------- oracle
    def oracle_ancestry(self, t: int) -> np.ndarray:
        return oracle.ancestry(self.parents, self.w.batch, self.w.beams, t)

    def oracle_request_head(self, q, b: int, hd: int, t: int) -> np.ndarray:
        """float64 [beams, D] for request b, head hd at step t, from a
        one-request one-head sub-problem cut out of the device tensors."""
        w = self.w
        W = w.beams
        kvh = hd // (w.heads // w.kv_heads)
        sl = slice(b * W, (b + 1) * W)
        qb = wl.to_bits(q[sl, hd:hd + 1])
        if self.kp is not None:
            n = self.kp.shape[1] if self.prompt_lens is None else self.prompt_lens[b]
            kpb = wl.to_bits(self.kp[b:b + 1, :n, kvh:kvh + 1]); vpb = wl.to_bits(self.vp[b:b + 1, :n, kvh:kvh + 1])
        else:
            kpb = vpb = np.zeros((1, 0, 1, w.head_dim), np.uint16)
        if t >= 0:
            krb = np.stack([wl.to_bits(k[sl, kvh:kvh + 1]) for k in self.k_steps[:t + 1]])
            vrb = np.stack([wl.to_bits(v[sl, kvh:kvh + 1]) for v in self.v_steps[:t + 1]])
            par = self.parents[:t + 1, sl]
        else:
            krb = vrb = par = None
        slopes = self.slopes[hd:hd + 1].cpu().numpy() if self.slopes is not None else None
        return oracle.decode_sdpa(w.dtype, 1, W, 1, 1, w.head_dim, qb, kpb, vpb, krb, vrb, par, t,
                                  slopes=slopes)[:, 0, :]

    def check(self, out, q, t: int, pairs):
        """Compare `out` with the oracle on (request, head) pairs; returns max abs error."""
        W = self.w.beams
        worst = 0.0
        for b, hd in pairs:
            ref = self.oracle_request_head(q, b, hd, t)
            got = out[b * W:(b + 1) * W, hd].to(torch.float64).cpu().numpy()
            assert np.isfinite(got).all(), f"non-finite output at request {b} head {hd}"
            err = np.abs(got - ref)
            bound = ATOL + RTOL * np.abs(ref)
            assert (err <= bound).all(), (
                f"request {b} head {hd} step {t}: max err {err.max():.3e}, worst excess {(err - bound).max():.3e}")
            worst = max(worst, float(err.max()))
        return worst


def all_pairs(w):
    return [(b, h) for b in range(w.batch) for h in range(w.heads)]


def sampled_pairs(w, n=64, seed=0):
    rng = np.random.default_rng(w.seed + seed)
    pairs = {(0, 0), (0, w.heads - 1), (w.batch - 1, 0), (w.batch - 1, w.heads - 1)}
    while len(pairs) < min(n + 4, w.batch * w.heads):
        pairs.add((int(rng.integers(w.batch)), int(rng.integers(w.heads))))
    return sorted(pairs)


def unique_rows_from_ancestry(anc: np.ndarray, batch: int, beams: int) -> np.ndarray:
    """[batch] distinct response rows per request, counted from a beam-index table."""
    out = np.zeros(batch, dtype=np.int64)
    for b in range(batch):
        blk = anc[b * beams:(b + 1) * beams]
        out[b] = sum(len(set(blk[:, s].tolist())) for s in range(anc.shape[1]))
    return out
