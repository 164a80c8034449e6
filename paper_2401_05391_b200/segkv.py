"""Thin ctypes binding of the segkv C-ABI (``include/segkv.h``).

Argument marshalling only: every step of the decode path runs in the library's
CUDA kernels.  PyTorch appears only as the owner of device memory and streams.
The module-level functions carry the C names; :class:`SegKV` wraps a handle.
There is no fallback: if ``libsegkv.so`` has not been built the import of the
library fails with an error that says how to build it.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsegkv.so")

SEGKV_F16, SEGKV_BF16 = 0, 1
SEGKV_OK, SEGKV_EINVAL, SEGKV_ESTATE, SEGKV_ECAPACITY, SEGKV_ENOMEM, SEGKV_ECUDA, SEGKV_EDEVICE = 0, -1, -2, -3, -4, -5, -6
SEGKV_DEV_BAD_PARENT, SEGKV_DEV_WAIT_LIMIT = 1, 2

_vp, _int, _i32p = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int32)

# name -> (restype, argtypes); one entry per symbol include/segkv.h declares
SIGNATURES = {
    "segkv_create": (_int, [ctypes.POINTER(_vp)] + [_int] * 8),
    "segkv_create_growing": (_int, [ctypes.POINTER(_vp)] + [_int] * 9),
    "segkv_allocated_kv_bytes": (ctypes.c_longlong, [_vp]),
    "segkv_destroy": (_int, [_vp]),
    "segkv_prefill_write": (_int, [_vp, _vp, _vp, _int, _vp]),
    "segkv_prefill_sdpa": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "segkv_prefill": (_int, [_vp, _vp, _vp, _vp, _vp, _int, _vp, _vp]),
    "segkv_append": (_int, [_vp, _int, _vp, _vp, _vp, _vp]),
    "segkv_decode_sdpa": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "segkv_decode_step": (_int, [_vp, _int, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "segkv_decode_sdpa_static": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "segkv_step_host": (_int, [_vp, _int, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "segkv_host_pack_bytes": (ctypes.c_size_t, [_vp, _vp]),
    "segkv_step_host_packed": (_int, [_vp, _int, _vp, _vp, _int, _vp]),
    "segkv_step_host_packed_async": (_int, [_vp, _int, _vp, _vp, _int, _vp]),
    "segkv_layers_step_host": (_int, [_vp, _int, _int, _vp, _vp, _int, _int, _vp]),
    "segkv_reset": (_int, [_vp, _int]),
    "segkv_truncate_last": (_int, [_vp]),
    "segkv_get_ancestry": (_int, [_vp, _vp, _vp]),
    "segkv_get_unique_rows": (_int, [_vp, _vp, _vp]),
    "segkv_get_error": (_int, [_vp, ctypes.POINTER(_int)]),
    "segkv_steps": (_int, [_vp]),
    "segkv_prompt_len": (_int, [_vp]),
    "segkv_set_tuning": (_int, [_vp, _int, _int, _int]),
    "segkv_set_tile": (_int, [_vp, _int]),
    "segkv_set_persistent": (_int, [_vp, _int]),
    "segkv_decode_sdpa_rowwise": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "segkv_get_splits": (_int, [_vp]),
    "segkv_set_overlap": (_int, [_vp, _int]),
    "segkv_set_prefill_tuning": (_int, [_vp, _int]),
    "segkv_set_prompt_layout": (_int, [_vp, _int]),
    "segkv_share_index": (_int, [_vp, _vp]),
    "segkv_append_rope": (_int, [_vp, _int, _vp, _vp, _vp, _vp, _vp, _int, _int, _vp]),
    "segkv_prefill_write_ragged": (_int, [_vp, _vp, _vp, _int, _vp, _vp]),
    "segkv_debug_inject": (_int, [_vp, ctypes.c_longlong, _int]),
    "segkv_read_bandwidth": (_int, [_vp, ctypes.c_size_t, _int, ctypes.POINTER(ctypes.c_float), _vp]),
    "segkv_launch_count": (ctypes.c_longlong, [_vp]),
    "segkv_storage_bytes": (ctypes.c_size_t, [_int] * 7),
    "segkv_strerror": (ctypes.c_char_p, [_int]),
    "segkv_last_cuda_error": (ctypes.c_char_p, []),
}

_lib = None


def lib() -> ctypes.CDLL:
    """Load ``libsegkv.so`` (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2401_05391_b200.build` "
                "(needs nvcc); there is no non-CUDA fallback")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class LayerStack:
    """The handles of a model's layers with their pinned host blocks, for segkv_layers_step_host."""

    def __init__(self, handles, packed_in, outs):
        n = len(handles)
        assert n == len(packed_in) == len(outs) and n > 0
        total = handles[0].host_pack_layout()[0]
        qs = (handles[0].rows, handles[0].heads, handles[0].head_dim)
        self._keep = (list(handles), list(packed_in), list(outs))
        self.n = n
        self._h = (_vp * n)(*[h._h for h in handles])
        self._in = (_vp * n)(*[_host(t, (total,), torch.uint8, "packed") for t in packed_in])
        self._out = (_vp * n)(*[_host(o, qs, handles[0].dtype, "out") for o in outs])

    def step(self, step: int, has_slopes: bool = False, redo: bool = False, stream=None) -> None:
        """Queue one decode step of every layer on the stream (the caller waits for the stream)."""
        _check(lib().segkv_layers_step_host(self._h, self.n, step, self._in, self._out, int(has_slopes), int(redo),
                                            _stream_ptr(stream)), "segkv_layers_step_host")


class SegKVError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().segkv_strerror(code).decode()
        if code == SEGKV_ECUDA:
            msg += ": " + lib().segkv_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({code})")


def _check(code: int, where: str) -> None:
    if code != SEGKV_OK:
        raise SegKVError(code, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dev(t: Optional[torch.Tensor], shape, dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected {tuple(shape)} {dtype}, got {tuple(t.shape)} {t.dtype}")
    return t.data_ptr()


def _host(t: Optional[torch.Tensor], shape, dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    if t.dtype != dtype or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected {tuple(shape)} {dtype}, got {tuple(t.shape)} {t.dtype}")
    return t.data_ptr()


def segkv_storage_bytes(batch, beams, kv_heads, head_dim, max_prompt, max_steps, dtype) -> int:
    return int(lib().segkv_storage_bytes(batch, beams, kv_heads, head_dim, max_prompt, max_steps, dtype))


def read_bandwidth(buf: torch.Tensor, repeats: int = 10, stream=None) -> float:
    """GB/s of a read-only pass over a CUDA tensor (segkv_read_bandwidth)."""
    if not buf.is_cuda or not buf.is_contiguous():
        raise ValueError("buf must be a contiguous CUDA tensor")
    gbs = ctypes.c_float(0)
    _check(lib().segkv_read_bandwidth(buf.data_ptr(), buf.numel() * buf.element_size(), repeats, ctypes.byref(gbs),
                                      _stream_ptr(stream)), "segkv_read_bandwidth")
    return float(gbs.value)


def segkv_strerror(code: int) -> str:
    return lib().segkv_strerror(code).decode()


class SegKV:
    """One attention layer's segment KV cache; methods mirror the C entry points."""

    def __init__(self, batch, beams, heads, kv_heads, head_dim, max_prompt, max_steps, dtype=torch.float16,
                 chunk_steps: int = 0):
        self.batch, self.beams, self.heads, self.kv_heads = batch, beams, heads, kv_heads
        self.head_dim, self.max_prompt, self.max_steps = head_dim, max_prompt, max_steps
        self.dtype = dtype
        self.rows = batch * beams
        code = {torch.float16: SEGKV_F16, torch.bfloat16: SEGKV_BF16}.get(dtype, -1)
        self._h = _vp()
        if chunk_steps:
            _check(lib().segkv_create_growing(ctypes.byref(self._h), batch, beams, heads, kv_heads, head_dim,
                                              max_prompt, max_steps, chunk_steps, code), "segkv_create_growing")
        else:
            _check(lib().segkv_create(ctypes.byref(self._h), batch, beams, heads, kv_heads, head_dim,
                                      max_prompt, max_steps, code), "segkv_create")

    # ------------------------------------------------------------ life cycle
    def destroy(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            _check(lib().segkv_destroy(self._h), "segkv_destroy")     # refused while other handles follow this one
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()

    # -------------------------------------------------------------- hot path
    def prefill_write(self, k: Optional[torch.Tensor], v: Optional[torch.Tensor], stream=None) -> None:
        p = 0 if k is None else int(k.shape[1])
        shape = (self.batch, p, self.kv_heads, self.head_dim)
        _check(lib().segkv_prefill_write(self._h, _dev(k, shape, self.dtype, "k"), _dev(v, shape, self.dtype, "v"),
                                         p, _stream_ptr(stream)), "segkv_prefill_write")

    def prefill_write_ragged(self, k: torch.Tensor, v: torch.Tensor, prompt_lens, stream=None) -> None:
        """k, v: [batch, padded_len, kv_heads, head_dim] on the device; prompt_lens: batch host integers."""
        p = int(k.shape[1])
        shape = (self.batch, p, self.kv_heads, self.head_dim)
        lens = (ctypes.c_int32 * self.batch)(*[int(x) for x in prompt_lens])
        if len(prompt_lens) != self.batch:
            raise ValueError("prompt_lens needs one entry per request")
        _check(lib().segkv_prefill_write_ragged(self._h, _dev(k, shape, self.dtype, "k"),
                                                _dev(v, shape, self.dtype, "v"), p,
                                                ctypes.cast(lens, ctypes.c_void_p), _stream_ptr(stream)),
               "segkv_prefill_write_ragged")

    def prefill_sdpa(self, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                     alibi_slopes: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        shape = (self.batch, self.prompt_len, self.heads, self.head_dim)
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=q.device)
        _check(lib().segkv_prefill_sdpa(self._h, _dev(q, shape, self.dtype, "q"), _dev(out, shape, self.dtype, "out"),
                                        _dev(alibi_slopes, (self.heads,), torch.float32, "alibi_slopes"),
                                        _stream_ptr(stream)), "segkv_prefill_sdpa")
        return out

    def prefill(self, k: torch.Tensor, v: torch.Tensor, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                alibi_slopes: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        p = int(k.shape[1])
        kv = (self.batch, p, self.kv_heads, self.head_dim)
        qs = (self.batch, p, self.heads, self.head_dim)
        if out is None:
            out = torch.empty(qs, dtype=self.dtype, device=q.device)
        _check(lib().segkv_prefill(self._h, _dev(k, kv, self.dtype, "k"), _dev(v, kv, self.dtype, "v"),
                                   _dev(q, qs, self.dtype, "q"), _dev(out, qs, self.dtype, "out"), p,
                                   _dev(alibi_slopes, (self.heads,), torch.float32, "alibi_slopes"),
                                   _stream_ptr(stream)), "segkv_prefill")
        return out

    def append(self, step: int, beam_parent: Optional[torch.Tensor], k_new: torch.Tensor, v_new: torch.Tensor,
               stream=None) -> None:
        shape = (self.rows, self.kv_heads, self.head_dim)
        _check(lib().segkv_append(self._h, step, _dev(beam_parent, (self.rows,), torch.int32, "beam_parent"),
                                  _dev(k_new, shape, self.dtype, "k_new"), _dev(v_new, shape, self.dtype, "v_new"),
                                  _stream_ptr(stream)), "segkv_append")

    ROPE_STYLES = {"half": 1, "interleaved": 2}

    def append_rope(self, step: int, beam_parent: Optional[torch.Tensor], k_new: torch.Tensor, v_new: torch.Tensor,
                    rope_cos: torch.Tensor, rope_sin: torch.Tensor, style="half", stream=None) -> None:
        """append() with the rotary embedding applied to the new K rows; rope_cos / rope_sin are
        device fp32 [positions, head_dim/2]."""
        shape = (self.rows, self.kv_heads, self.head_dim)
        n = int(rope_cos.shape[0])
        tshape = (n, self.head_dim // 2)
        code = self.ROPE_STYLES[style] if isinstance(style, str) else int(style)
        _check(lib().segkv_append_rope(self._h, step, _dev(beam_parent, (self.rows,), torch.int32, "beam_parent"),
                                       _dev(k_new, shape, self.dtype, "k_new"), _dev(v_new, shape, self.dtype, "v_new"),
                                       _dev(rope_cos, tshape, torch.float32, "rope_cos"),
                                       _dev(rope_sin, tshape, torch.float32, "rope_sin"), n, code,
                                       _stream_ptr(stream)), "segkv_append_rope")

    def decode_sdpa(self, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                    alibi_slopes: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        shape = (self.rows, self.heads, self.head_dim)
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=q.device)
        _check(lib().segkv_decode_sdpa(self._h, _dev(q, shape, self.dtype, "q"), _dev(out, shape, self.dtype, "out"),
                                       _dev(alibi_slopes, (self.heads,), torch.float32, "alibi_slopes"),
                                       _stream_ptr(stream)), "segkv_decode_sdpa")
        return out

    def decode_step(self, step: int, beam_parent: Optional[torch.Tensor], k_new: torch.Tensor, v_new: torch.Tensor,
                    q: torch.Tensor, out: Optional[torch.Tensor] = None,
                    alibi_slopes: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        kv = (self.rows, self.kv_heads, self.head_dim)
        qs = (self.rows, self.heads, self.head_dim)
        if out is None:
            out = torch.empty(qs, dtype=self.dtype, device=q.device)
        _check(lib().segkv_decode_step(self._h, step, _dev(beam_parent, (self.rows,), torch.int32, "beam_parent"),
                                       _dev(k_new, kv, self.dtype, "k_new"), _dev(v_new, kv, self.dtype, "v_new"),
                                       _dev(q, qs, self.dtype, "q"), _dev(out, qs, self.dtype, "out"),
                                       _dev(alibi_slopes, (self.heads,), torch.float32, "alibi_slopes"),
                                       _stream_ptr(stream)), "segkv_decode_step")
        return out

    def decode_sdpa_static(self, q: torch.Tensor, out: torch.Tensor,
                           alibi_slopes: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """segkv_decode_sdpa_static: same attention, split workspace in the library's built-in
        device array, no allocation by the library (``out`` must be given for the same reason)."""
        shape = (self.rows, self.heads, self.head_dim)
        _check(lib().segkv_decode_sdpa_static(self._h, _dev(q, shape, self.dtype, "q"),
                                              _dev(out, shape, self.dtype, "out"),
                                              _dev(alibi_slopes, (self.heads,), torch.float32, "alibi_slopes"),
                                              _stream_ptr(stream)), "segkv_decode_sdpa_static")
        return out

    def step_host(self, step: int, beam_parent, k_new, v_new, q, out, alibi_slopes=None, stream=None) -> torch.Tensor:
        kv = (self.rows, self.kv_heads, self.head_dim)
        qs = (self.rows, self.heads, self.head_dim)
        _check(lib().segkv_step_host(self._h, step, _host(beam_parent, (self.rows,), torch.int32, "beam_parent"),
                                     _host(k_new, kv, self.dtype, "k_new"), _host(v_new, kv, self.dtype, "v_new"),
                                     _host(q, qs, self.dtype, "q"), _host(out, qs, self.dtype, "out"),
                                     _host(alibi_slopes, (self.heads,), torch.float32, "alibi_slopes"),
                                     _stream_ptr(stream)), "segkv_step_host")
        return out

    def host_pack_layout(self):
        """(total bytes, offsets of beam_parent / slopes / k_new / v_new / q) of the packed host block."""
        off = (ctypes.c_size_t * 5)()
        total = int(lib().segkv_host_pack_bytes(self._h, ctypes.cast(off, ctypes.c_void_p)))
        return total, [int(x) for x in off]

    def step_host_packed(self, step: int, packed: torch.Tensor, out: torch.Tensor, has_slopes: bool = False,
                         stream=None) -> torch.Tensor:
        """One step from one packed host block (a uint8 tensor laid out as host_pack_layout says)."""
        total, _ = self.host_pack_layout()
        qs = (self.rows, self.heads, self.head_dim)
        _check(lib().segkv_step_host_packed(self._h, step, _host(packed, (total,), torch.uint8, "packed"),
                                            _host(out, qs, self.dtype, "out"), int(has_slopes), _stream_ptr(stream)),
               "segkv_step_host_packed")
        return out

    def step_host_packed_async(self, step: int, packed: torch.Tensor, out: torch.Tensor, has_slopes: bool = False,
                               stream=None) -> torch.Tensor:
        """As step_host_packed, but only queued on the stream: wait for the stream before reading `out`."""
        if getattr(self, "_pack_total", None) is None:
            self._pack_total = self.host_pack_layout()[0]
        qs = (self.rows, self.heads, self.head_dim)
        _check(lib().segkv_step_host_packed_async(self._h, step, _host(packed, (self._pack_total,), torch.uint8, "packed"),
                                                  _host(out, qs, self.dtype, "out"), int(has_slopes),
                                                  _stream_ptr(stream)),
               "segkv_step_host_packed_async")
        return out

    # ------------------------------------------------------------------ aids
    def reset(self, keep_prompt: bool = True) -> None:
        _check(lib().segkv_reset(self._h, int(keep_prompt)), "segkv_reset")

    def truncate_last(self) -> None:
        _check(lib().segkv_truncate_last(self._h), "segkv_truncate_last")

    @property
    def steps(self) -> int:
        return int(lib().segkv_steps(self._h))

    @property
    def prompt_len(self) -> int:
        return int(lib().segkv_prompt_len(self._h))

    def get_ancestry(self, stream=None) -> np.ndarray:
        out = np.empty((self.rows, self.steps), dtype=np.int32)
        _check(lib().segkv_get_ancestry(self._h, out.ctypes.data, _stream_ptr(stream)), "segkv_get_ancestry")
        return out

    def get_unique_rows(self, stream=None) -> np.ndarray:
        out = np.empty((self.batch,), dtype=np.int32)
        _check(lib().segkv_get_unique_rows(self._h, out.ctypes.data, _stream_ptr(stream)), "segkv_get_unique_rows")
        return out

    def get_error(self) -> int:
        flags = _int(0)
        _check(lib().segkv_get_error(self._h, ctypes.byref(flags)), "segkv_get_error")
        return flags.value

    def set_tile(self, tile_keys: int = 0) -> None:
        _check(lib().segkv_set_tile(self._h, tile_keys), "segkv_set_tile")

    def set_persistent(self, mode):
        _check(lib().segkv_set_persistent(self._h, mode), "segkv_set_persistent")

    def debug_inject(self, wait_limit_ns: int = 0, skip_arrival: bool = False) -> None:
        _check(lib().segkv_debug_inject(self._h, int(wait_limit_ns), int(bool(skip_arrival))), "segkv_debug_inject")

    def set_tuning(self, splits: int = 0, stages: int = 0, combine: int = 0) -> None:
        _check(lib().segkv_set_tuning(self._h, splits, stages, combine), "segkv_set_tuning")

    def decode_sdpa_rowwise(self, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                            alibi_slopes: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        shape = (self.rows, self.heads, self.head_dim)
        if out is None:
            out = torch.empty(shape, dtype=self.dtype, device=q.device)
        _check(lib().segkv_decode_sdpa_rowwise(self._h, _dev(q, shape, self.dtype, "q"),
                                               _dev(out, shape, self.dtype, "out"),
                                               _dev(alibi_slopes, (self.heads,), torch.float32, "alibi_slopes"),
                                               _stream_ptr(stream)), "segkv_decode_sdpa_rowwise")
        return out

    def set_overlap(self, enable: bool) -> None:
        _check(lib().segkv_set_overlap(self._h, int(enable)), "segkv_set_overlap")

    def share_index(self, leader: Optional["SegKV"]) -> None:
        """Use `leader`'s beam-index tables (one table for all layers of a model); None undoes it."""
        _check(lib().segkv_share_index(self._h, None if leader is None else leader._h), "segkv_share_index")

    PROMPT_LAYOUTS = {"head_major": 0, "token_major": 1, "seq_first": 2}

    def set_prompt_layout(self, layout) -> None:
        code = self.PROMPT_LAYOUTS[layout] if isinstance(layout, str) else int(layout)
        _check(lib().segkv_set_prompt_layout(self._h, code), "segkv_set_prompt_layout")

    def set_prefill_tuning(self, row_groups: int = 0) -> None:
        _check(lib().segkv_set_prefill_tuning(self._h, row_groups), "segkv_set_prefill_tuning")

    def get_splits(self) -> int:
        return int(lib().segkv_get_splits(self._h))

    @property
    def allocated_kv_bytes(self) -> int:
        return int(lib().segkv_allocated_kv_bytes(self._h))

    @property
    def launch_count(self) -> int:
        return int(lib().segkv_launch_count(self._h))
