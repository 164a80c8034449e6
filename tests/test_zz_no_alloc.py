"""The allocation-free attention entry point (collected last on purpose).

Some callers of this library cannot let it allocate device memory in the decode
loop: a server whose memory pool already owns the whole GPU, a loop that must not
stall behind the device-wide synchronisation of an allocation, a plug-in that is
forbidden to call the CUDA allocator.  ``segkv_decode_sdpa_static`` serves them
by keeping the split workspace in an array built into the library.  The test
calls it through the C-ABI twice in a row (the array is shared and keeps the
previous call's contents, so the second call proves it is cleared correctly) and
checks it against the regular entry point.
"""
import ctypes

import pytest
import torch

from paper_2401_05391_b200 import segkv as sk
from paper_2401_05391_b200 import workloads as wl

from _harness import ATOL, RTOL, Run, all_pairs

pytestmark = pytest.mark.gpu


def _close(a, b):
    a, b = a.double(), b.double()
    return bool(((a - b).abs() <= ATOL + RTOL * b.abs()).all())


def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row():
    w = wl.CONFIGS[1].scaled(steps=24, index=50)            # 32 work groups -> several splits each
    r = Run(w)
    try:
        r.advance_to(w.steps - 1)
        assert r.h.get_splits() > 1
        ref, q = r.decode()
        lib = sk.lib()
        stream = torch.cuda.current_stream().cuda_stream
        for call in range(2):
            out = torch.full_like(ref, float("nan"))
            rc = lib.segkv_decode_sdpa_static(r.h._h, ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(out.data_ptr()),
                                              None, ctypes.c_void_p(stream))
            assert rc == sk.SEGKV_OK, sk.segkv_strerror(rc)
            torch.cuda.synchronize()
            assert not torch.isnan(out.float()).any(), f"call {call}: unwritten outputs"
            assert _close(out, ref), f"call {call}: differs from segkv_decode_sdpa beyond the tolerance"
            r.check(out, q, w.steps - 1, all_pairs(w))             # and against the CPU oracle itself
        # a different split count right after: other ticket/partial footprint in the same array
        r.h.set_tuning(3, 0, 0)
        out = torch.full_like(ref, float("nan"))
        r.h.decode_sdpa_static(q, out)
        torch.cuda.synchronize()
        assert _close(out, ref)
        assert r.h.get_error() == 0
    finally:
        r.close()


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    # 512 work groups x 64 splits x 4 columns x 130 floats = 68 MB of partials: beyond the built-in 8 MiB
    w = wl.Workload("big", 32, 4, 16, 16, 128, 4096, 2, "f16", "uniform", False, 51)
    h = sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype)
    try:
        kp, vp = wl.make_prompt(w, "cuda")
        h.prefill_write(kp, vp)
        q = torch.zeros(w.rows, w.heads, w.head_dim, dtype=torch.float16, device="cuda")
        out = torch.zeros_like(q)
        h.set_tuning(64, 0, 0)
        with pytest.raises(sk.SegKVError) as e:
            h.decode_sdpa_static(q, out)
        assert e.value.code == sk.SEGKV_ECAPACITY
        h.set_tuning(1, 0, 0)                               # one split needs no scratch at all
        h.decode_sdpa_static(q, out)
        torch.cuda.synchronize()
    finally:
        h.destroy()


def test_static_scratch_entry_point_checks_the_shared_index_tables_step():
    # a handle that reads another handle's beam-index tables must be at the leader's step, as for
    # segkv_decode_sdpa: after the leader has moved on, its tables describe another step
    w = wl.Workload("follow", 1, 4, 4, 4, 128, 64, 4, "f16", "uniform", False, 52)
    lead = Run(w)
    foll = Run(w.scaled(index=53), parents=lead.parents)
    try:
        foll.h.share_index(lead.h)
        for _ in range(2):
            lead.append_next(); foll.append_next()
        q = foll.q_steps[-1]
        out = torch.full((w.rows, w.heads, w.head_dim), float("nan"), dtype=w.torch_dtype, device="cuda")
        foll.h.decode_sdpa_static(q, out)                       # same step: fine
        torch.cuda.synchronize()
        foll.check(out, q, 1, all_pairs(w))
        lead.append_next()                                      # the leader moves on alone
        with pytest.raises(sk.SegKVError) as e:
            foll.h.decode_sdpa_static(q, out)
        assert e.value.code == sk.SEGKV_ESTATE
    finally:
        foll.close(); lead.close()
