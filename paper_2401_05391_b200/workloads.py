"""Seeded synthetic workloads for the segment-KV decode attention path.

This module only *describes* and *draws* inputs: tensor shapes, value
distributions, beam-parent tables and ALiBi slope vectors.  It contains none of
the attention / ancestry arithmetic, so both the CUDA path and the CPU oracle
can be fed from it without sharing any of the method's code.

The paper evaluates on fixed-length prompts (N_prompt = 1024, N_response = 128,
fp16, beam width 4; Section 4) pushed through real LLMs.  Neither weights nor a
beam-search module exist here, so activations are iid N(0,1) values rounded to
the storage dtype (RoPE assumed already applied) and the per-step beam parents
are seeded random draws.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import numpy as np
import torch

BASE_SEED = 20240105


@dataclass(frozen=True)
class Workload:
    """One attention-layer decode workload (paper notation in brackets)."""

    name: str
    batch: int          # BS
    beams: int          # BW
    heads: int          # H (query heads)
    kv_heads: int       # key/value heads (== heads for the paper's MHA models)
    head_dim: int       # D
    prompt_len: int     # N_prompt
    steps: int          # N_response
    dtype: str          # "f16" | "bf16"
    parents: str        # "uniform" | "half_identity"
    alibi: bool
    index: int          # position in the config list; seeds derive from it

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float16 if self.dtype == "f16" else torch.bfloat16

    @property
    def rows(self) -> int:
        """Number of beam slots, BS x BW."""
        return self.batch * self.beams

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five evaluation shapes: a tiny case, then the attention-layer shapes of
# Llama2-7B, GPT-J-6B (16 heads x 256), OPT-30B and Bloom-176B (ALiBi, bf16).
CONFIGS = (
    Workload("tiny", 1, 4, 4, 4, 64, 32, 8, "f16", "uniform", False, 0),
    Workload("llama2-7b", 1, 4, 32, 32, 128, 1024, 128, "f16", "uniform", False, 1),
    Workload("gptj-6b", 16, 4, 16, 16, 256, 1024, 128, "f16", "uniform", False, 2),
    Workload("opt-30b", 64, 4, 56, 56, 128, 2048, 256, "f16", "half_identity", False, 3),
    Workload("bloom-176b", 32, 4, 112, 112, 128, 1024, 128, "bf16", "uniform", True, 4),
)
# The shape of the paper's own kernel experiment (Section 4.1, Fig. 6).
LLAMA2_13B = Workload("llama2-13b", 1, 4, 40, 40, 128, 1024, 128, "f16", "uniform", False, 5)


def by_name(name: str) -> Workload:
    for c in CONFIGS + (LLAMA2_13B,):
        if c.name == name:
            return c
    raise KeyError(name)


def make_parents(w: Workload, seed: Optional[int] = None) -> np.ndarray:
    """Beam-parent table ``[steps, batch*beams]`` int32 with LOCAL ids in [0, beams).

    ``parent[s, b*beams + j]`` names the beam slot (within request b) at step
    s-1 that slot j extends at step s.  Row 0 is drawn too but has no meaning
    (every beam descends from the shared prompt).

    "uniform": every entry iid uniform.  "half_identity": per (request, step) a
    fair coin keeps every beam on its own slot, else the row is iid uniform.
    """
    rng = np.random.default_rng(w.seed if seed is None else seed)
    par = rng.integers(0, w.beams, size=(w.steps, w.batch, w.beams), dtype=np.int64)
    if w.parents == "half_identity":
        keep = rng.random(size=(w.steps, w.batch)) < 0.5
        ident = np.broadcast_to(np.arange(w.beams), par.shape)
        par = np.where(keep[:, :, None], ident, par)
    elif w.parents != "uniform":
        raise ValueError(w.parents)
    return np.ascontiguousarray(par.reshape(w.steps, w.rows).astype(np.int32))


def alibi_slopes(heads: int) -> torch.Tensor:
    """fp32 slope vector ``2^(-8 i / heads)``, i = 1..heads (the Bloom config's recipe)."""
    i = torch.arange(1, heads + 1, dtype=torch.float64)
    return torch.pow(torch.tensor(2.0, dtype=torch.float64), -8.0 * i / heads).to(torch.float32)


def rope_tables(positions: int, head_dim: int, base: float = 10000.0):
    """fp32 tables cos / sin [positions, head_dim/2] of the angle ``m * base^(-2i/head_dim)`` for
    position m and pair i: the input a rotary-embedding kernel is given (computed in float64,
    rounded once)."""
    m = torch.arange(positions, dtype=torch.float64)[:, None]
    i = torch.arange(head_dim // 2, dtype=torch.float64)[None, :]
    ang = m * torch.pow(torch.tensor(float(base), dtype=torch.float64), -2.0 * i / head_dim)
    return torch.cos(ang).to(torch.float32), torch.sin(ang).to(torch.float32)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _normal(shape, w: Workload, device, seed: int) -> torch.Tensor:
    # drawn in fp32, then rounded once to the storage dtype
    x = torch.randn(shape, generator=_gen(device, seed), device=device, dtype=torch.float32)
    return x.to(w.torch_dtype)


def make_prompt(w: Workload, device="cpu", prompt_len: Optional[int] = None):
    """Prompt K and V, token-major ``[batch, prompt_len, kv_heads, head_dim]``
    (the layout a fused QKV projection emits at prefill)."""
    p = w.prompt_len if prompt_len is None else prompt_len
    shape = (w.batch, p, w.kv_heads, w.head_dim)
    return (_normal(shape, w, device, w.seed * 1000 + 1),
            _normal(shape, w, device, w.seed * 1000 + 2))


def make_prefill_query(w: Workload, device="cpu", prompt_len: Optional[int] = None) -> torch.Tensor:
    """Prefill queries, token-major ``[batch, prompt_len, heads, head_dim]``."""
    p = w.prompt_len if prompt_len is None else prompt_len
    return _normal((w.batch, p, w.heads, w.head_dim), w, device, w.seed * 1000 + 3)


def make_step(w: Workload, step: int, device="cpu"):
    """Step ``step``'s q ``[rows, heads, D]`` and new k, v ``[rows, kv_heads, D]``.

    Each step has its own seed so any step can be re-drawn on its own."""
    base = w.seed * 1000 + 10 + 3 * step
    q = _normal((w.rows, w.heads, w.head_dim), w, device, base)
    k = _normal((w.rows, w.kv_heads, w.head_dim), w, device, base + 1)
    v = _normal((w.rows, w.kv_heads, w.head_dim), w, device, base + 2)
    return q, k, v


def to_bits(t: torch.Tensor) -> np.ndarray:
    """The raw 16-bit patterns of an fp16/bf16 tensor as a host uint16 array."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
