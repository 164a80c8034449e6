"""CPU float64 oracle for the segment-KV decode attention path (Python face).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg, never by the product package.  The arithmetic is
in ``segkv_oracle.c`` (plain C, double precision, one OpenMP loop over output
rows); this file compiles it with the host compiler and marshals numpy arrays.

Parity status: the attention context has no printed value in the paper, so it
is pinned by special cases, closed forms, invariants and a copied-cache brute
force (``tests/test_oracle_pins.py``); the cache-size formulas are pinned to
the values the paper prints for GPT-J-6B (Section 3.2); the rotary embedding
of key rows (``rope``, numpy float64) is pinned to complex multiplication, the
identity at position 0, the exact quarter turn, norm preservation and the
relative-position property, and ``narrow`` to torch's conversions.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "segkv_oracle.c")
_LIB = os.path.join(_HERE, "libsegkv_oracle.so")
_lib = None

F16, BF16 = 0, 1
DTYPES = {"f16": F16, "bf16": BF16}


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no GPU toolchain involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        f64p = ctypes.POINTER(ctypes.c_double)
        f32p = ctypes.POINTER(ctypes.c_float)
        c_int = ctypes.c_int
        lib.segkv_oracle_widen.argtypes = [c_int, u16p, ctypes.c_long, f64p]
        lib.segkv_oracle_widen.restype = None
        lib.segkv_oracle_ancestry.argtypes = [i32p, c_int, c_int, c_int, i32p]
        lib.segkv_oracle_ancestry.restype = None
        lib.segkv_oracle_decode.argtypes = [c_int] * 8 + [u16p] * 5 + [i32p, f32p, i32p, c_int, f64p, f64p]
        lib.segkv_oracle_decode.restype = c_int
        lib.segkv_oracle_prefill.argtypes = [c_int] * 6 + [u16p] * 3 + [f32p, i32p, c_int, f64p]
        lib.segkv_oracle_prefill.restype = c_int
        lib.segkv_oracle_cache_token.argtypes = [c_int] * 4
        lib.segkv_oracle_cache_token.restype = ctypes.c_double
        lib.segkv_oracle_cache_standard.argtypes = [c_int, c_int, ctypes.c_long, ctypes.c_long, ctypes.c_double]
        lib.segkv_oracle_cache_standard.restype = ctypes.c_double
        lib.segkv_oracle_cache_segment.argtypes = [c_int, c_int, ctypes.c_long, ctypes.c_long, c_int, ctypes.c_double]
        lib.segkv_oracle_cache_segment.restype = ctypes.c_double
        lib.segkv_oracle_threads.restype = c_int
        _lib = lib
    return _lib


def _ptr(a: Optional[np.ndarray], ctype):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _u16(a, shape) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("16-bit storage must be passed as raw uint16 bit patterns")
    if tuple(a.shape) != tuple(shape):
        raise ValueError(f"shape {a.shape} != expected {tuple(shape)}")
    return a


def widen(dtype: str, bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().segkv_oracle_widen(DTYPES[dtype], _ptr(bits, ctypes.c_uint16), bits.size, _ptr(out, ctypes.c_double))
    return out


def ancestry(parent: np.ndarray, batch: int, beams: int, t: int) -> np.ndarray:
    """Beam-index table ``[batch*beams, t+1]`` at step t from parents ``[>=t+1, batch*beams]``."""
    parent = np.ascontiguousarray(parent, dtype=np.int32)
    if parent.ndim != 2 or parent.shape[1] != batch * beams or parent.shape[0] < t + 1:
        raise ValueError("parent must be [steps, batch*beams] with steps > t")
    if parent[1:t + 1].size and (parent[1:t + 1].min() < 0 or parent[1:t + 1].max() >= beams):
        raise ValueError("parent ids must be local, in [0, beams)")
    rows = np.empty((batch * beams, t + 1), dtype=np.int32)
    _load().segkv_oracle_ancestry(_ptr(parent, ctypes.c_int32), batch, beams, t, _ptr(rows, ctypes.c_int32))
    return rows


def decode_sdpa(dtype: str, batch: int, beams: int, heads: int, kv_heads: int, head_dim: int,
                q: np.ndarray, kp: np.ndarray, vp: np.ndarray,
                kr: Optional[np.ndarray], vr: Optional[np.ndarray], parent: Optional[np.ndarray],
                t: int, slopes: Optional[np.ndarray] = None,
                pairs: Optional[Sequence] = None, return_probs: bool = False):
    """Attention context at step ``t`` (``t = -1``: prompt only).

    q ``[rows, heads, D]``; kp, vp ``[batch, P, kv_heads, D]``; kr, vr
    ``[>=t+1, rows, kv_heads, D]``; parent ``[>=t+1, rows]`` (all uint16 bits
    except parent).  ``pairs`` = list of (g, h) to evaluate (default: all).
    Returns float64 ``[npairs, D]`` (reshaped to ``[rows, heads, D]`` when all
    pairs are asked for), plus the softmax rows when ``return_probs``.
    """
    rows = batch * beams
    P = int(kp.shape[1])
    q = _u16(q, (rows, heads, head_dim))
    kp = _u16(kp, (batch, P, kv_heads, head_dim))
    vp = _u16(vp, (batch, P, kv_heads, head_dim))
    if t >= 0:
        kr = _u16(np.asarray(kr)[:t + 1], (t + 1, rows, kv_heads, head_dim))
        vr = _u16(np.asarray(vr)[:t + 1], (t + 1, rows, kv_heads, head_dim))
        parent = np.ascontiguousarray(np.asarray(parent)[:t + 1], dtype=np.int32)
        if parent.shape != (t + 1, rows):
            raise ValueError("parent must be [steps, batch*beams]")
        if t >= 1 and (parent[1:].min() < 0 or parent[1:].max() >= beams):
            raise ValueError("parent ids must be local, in [0, beams)")
    else:
        kr = vr = parent = None
    if slopes is not None:
        slopes = np.ascontiguousarray(slopes, dtype=np.float32)
        if slopes.shape != (heads,):
            raise ValueError("slopes must be [heads]")
    all_pairs = pairs is None
    if all_pairs:
        gg, hh = np.meshgrid(np.arange(rows), np.arange(heads), indexing="ij")
        pairs_a = np.stack([gg.ravel(), hh.ravel()], axis=1)
    else:
        pairs_a = np.asarray(pairs).reshape(-1, 2)
    pairs_a = np.ascontiguousarray(pairs_a, dtype=np.int32)
    n = pairs_a.shape[0]
    L = P + t + 1
    out = np.empty((n, head_dim), dtype=np.float64)
    probs = np.empty((n, L), dtype=np.float64) if return_probs else None
    rc = _load().segkv_oracle_decode(
        DTYPES[dtype], batch, beams, heads, kv_heads, head_dim, P, t,
        _ptr(q, ctypes.c_uint16), _ptr(kp, ctypes.c_uint16), _ptr(vp, ctypes.c_uint16),
        _ptr(kr, ctypes.c_uint16), _ptr(vr, ctypes.c_uint16), _ptr(parent, ctypes.c_int32),
        _ptr(slopes, ctypes.c_float), _ptr(pairs_a, ctypes.c_int32), n,
        _ptr(out, ctypes.c_double), _ptr(probs, ctypes.c_double))
    if rc != 0:
        raise ValueError("segkv_oracle_decode rejected its arguments")
    if all_pairs:
        out = out.reshape(rows, heads, head_dim)
        if return_probs:
            probs = probs.reshape(rows, heads, L)
    return (out, probs) if return_probs else out


def prefill_sdpa(dtype: str, batch: int, heads: int, kv_heads: int, head_dim: int, q: np.ndarray, k: np.ndarray,
                 v: np.ndarray, slopes: Optional[np.ndarray] = None, rows: Optional[Sequence] = None) -> np.ndarray:
    """Causal prefill attention.  q ``[batch, N, heads, D]``, k, v ``[batch, N, kv_heads, D]`` (uint16
    bits).  ``rows`` = list of (b, i, h) to evaluate (default: all); returns float64 ``[nrows, D]``
    (``[batch, N, heads, D]`` when all rows are asked for)."""
    N = int(q.shape[1])
    q = _u16(q, (batch, N, heads, head_dim))
    k = _u16(k, (batch, N, kv_heads, head_dim))
    v = _u16(v, (batch, N, kv_heads, head_dim))
    if slopes is not None:
        slopes = np.ascontiguousarray(slopes, dtype=np.float32)
        if slopes.shape != (heads,):
            raise ValueError("slopes must be [heads]")
    all_rows = rows is None
    if all_rows:
        bb, ii, hh = np.meshgrid(np.arange(batch), np.arange(N), np.arange(heads), indexing="ij")
        rows_a = np.stack([bb.ravel(), ii.ravel(), hh.ravel()], axis=1)
    else:
        rows_a = np.asarray(rows).reshape(-1, 3)
    rows_a = np.ascontiguousarray(rows_a, dtype=np.int32)
    out = np.empty((rows_a.shape[0], head_dim), dtype=np.float64)
    rc = _load().segkv_oracle_prefill(DTYPES[dtype], batch, N, heads, kv_heads, head_dim,
                                      _ptr(q, ctypes.c_uint16), _ptr(k, ctypes.c_uint16), _ptr(v, ctypes.c_uint16),
                                      _ptr(slopes, ctypes.c_float), _ptr(rows_a, ctypes.c_int32), rows_a.shape[0],
                                      _ptr(out, ctypes.c_double))
    if rc != 0:
        raise ValueError("segkv_oracle_prefill rejected its arguments")
    return out.reshape(batch, N, heads, head_dim) if all_rows else out


def narrow(dtype: str, x: np.ndarray) -> np.ndarray:
    """float64 -> fp16 / bf16 bit patterns (uint16), round to nearest even.  bf16 goes through
    float32 first; the double rounding can only matter within 2^-24 of a bf16 tie."""
    x = np.asarray(x, np.float64)
    if dtype == "f16":
        return x.astype(np.float16).view(np.uint16)
    u = x.astype(np.float32).view(np.uint32).astype(np.uint64)
    return ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)


def rope(dtype: str, x: np.ndarray, cos: np.ndarray, sin: np.ndarray, style: str) -> np.ndarray:
    """Rotary position embedding of key rows (Section 3.1 lists a fused RoPE kernel; the rotation
    is the standard one): x [n, D] as bit patterns, cos / sin [n, D/2] the values for each row's
    position.  Pair i is (x[i], x[i + D/2]) for style "half" (Llama, NeoX) and (x[2i], x[2i+1])
    for style "interleaved" (GPT-J); each pair (a, b) becomes (a cos - b sin, b cos + a sin).
    Computed in float64, rounded once to the 16-bit type; returns bit patterns [n, D]."""
    xb = np.ascontiguousarray(x, np.uint16)
    n, D = xb.shape
    xf = widen(dtype, xb).reshape(n, D)
    c = np.asarray(cos, np.float64).reshape(n, D // 2)
    s = np.asarray(sin, np.float64).reshape(n, D // 2)
    out = np.empty_like(xf)
    if style == "half":
        a, b = xf[:, :D // 2], xf[:, D // 2:]
        out[:, :D // 2] = a * c - b * s
        out[:, D // 2:] = b * c + a * s
    elif style == "interleaved":
        a, b = xf[:, 0::2], xf[:, 1::2]
        out[:, 0::2] = a * c - b * s
        out[:, 1::2] = b * c + a * s
    else:
        raise ValueError(style)
    return narrow(dtype, out)


def cache_token(layers: int, heads: int, head_dim: int, elem_bytes: int) -> float:
    """Eq. 1: K and V bytes of one token over all layers."""
    return _load().segkv_oracle_cache_token(layers, heads, head_dim, elem_bytes)


def cache_standard(batch: int, beams: int, n_prompt: int, n_response: int, token: float) -> float:
    """Eq. 2: contiguous per-beam cache."""
    return _load().segkv_oracle_cache_standard(batch, beams, n_prompt, n_response, token)


def cache_segment(batch: int, beams: int, n_prompt: int, n_response: int, token: float, chunk: int = 16) -> float:
    """Eq. 3: segment cache with response capacity rounded up to ``chunk`` steps."""
    return _load().segkv_oracle_cache_segment(batch, beams, n_prompt, n_response, chunk, token)


def threads() -> int:
    return _load().segkv_oracle_threads()
