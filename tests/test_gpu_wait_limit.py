"""A bounded wait inside a kernel that runs out: the kernel must return by itself, report
SEGKV_DEV_WAIT_LIMIT, leave the output untouched, and leave the handle fit for the next call.

Nothing on a healthy device makes a wait run out, so the tests ask for it through
``segkv_debug_inject``: the next launch uses a 1 ms limit and one role leaves out one plain
mbarrier arrival (never a copy).  No trap, no unbounded loop, no bad address is involved."""
import numpy as np
import pytest
import torch

import oracle
from paper_2401_05391_b200 import segkv as sk
from paper_2401_05391_b200 import workloads as wl

from _harness import ATOL, RTOL, Run, all_pairs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("form", ["separate", "fused", "static", "persistent"])
@pytest.mark.parametrize("splits", [1, 3])
def test_decode_wait_runs_out_and_the_handle_recovers(form, splits):
    w = wl.Workload("wait", 2, 4, 4, 2, 128, 100, 6, "f16", "uniform", False, 71)
    r = Run(w, splits=splits, persistent=1 if form == "persistent" else -1)
    try:
        r.advance_to(3)
        if form == "fused":
            # the faulty launch is the fused step that appends step 4
            t = r.h.steps
            q, k, v = wl.make_step(w, t, "cuda")
            out = torch.full((w.rows, w.heads, w.head_dim), float("nan"), dtype=w.torch_dtype, device="cuda")
            r.h.debug_inject(1_000_000, True)
            r.h.decode_step(t, r.parents_dev[t], k, v, q, out)
            r.k_steps.append(k); r.v_steps.append(v); r.q_steps.append(q)
        else:
            q = r.q_steps[-1]
            out = torch.full((w.rows, w.heads, w.head_dim), float("nan"), dtype=w.torch_dtype, device="cuda")
            r.h.debug_inject(1_000_000, True)
            (r.h.decode_sdpa_static if form == "static" else r.h.decode_sdpa)(q, out)
        torch.cuda.synchronize()                                   # the kernel came back on its own
        assert r.h.get_error() & sk.SEGKV_DEV_WAIT_LIMIT
        assert torch.isnan(out.float()).all(), "a launch that gave up must not write the output"
        # the very next launches on the same handle are normal: same split count, so the work groups'
        # arrival counters must have come back to zero
        t = r.h.steps - 1
        for _ in range(2):
            out2, q2 = r.decode()
            r.check(out2, q2, t, all_pairs(w))
        _, out3, q3 = r.step_fused()
        r.check(out3, q3, t + 1, all_pairs(w))
        assert np.array_equal(r.h.get_ancestry(), r.oracle_ancestry(t + 1))
        assert r.h.get_error() == 0
    finally:
        r.close()


@pytest.mark.parametrize("D,groups", [(128, 1), (128, 2), (256, 0)])
def test_prefill_wait_runs_out_and_the_handle_recovers(D, groups):
    w = wl.Workload("waitpf", 1, 2, 2, 2, D, 300, 2, "f16", "uniform", False, 72)
    h = sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype)
    try:
        h.set_prefill_tuning(groups)
        kp, vp = wl.make_prompt(w, "cuda")
        q = wl.make_prefill_query(w, "cuda")
        h.prefill_write(kp, vp)
        out = torch.full_like(q, float("nan"))
        h.debug_inject(1_000_000, True)
        h.prefill_sdpa(q, out)
        torch.cuda.synchronize()
        assert h.get_error() & sk.SEGKV_DEV_WAIT_LIMIT
        assert torch.isnan(out.float()).all()
        out = torch.full_like(q, float("nan"))
        h.prefill_sdpa(q, out)                                       # tensor memory was released: the next launch runs
        torch.cuda.synchronize()
        rows = [(0, i, hd) for i in (0, 1, 127, 128, 299) for hd in range(w.heads)]
        ref = oracle.prefill_sdpa(w.dtype, w.batch, w.heads, w.kv_heads, w.head_dim, wl.to_bits(q), wl.to_bits(kp),
                                  wl.to_bits(vp), slopes=None, rows=rows)
        got = np.stack([out[b, i, hd].to(torch.float64).cpu().numpy() for b, i, hd in rows])
        assert (np.abs(got - ref) <= ATOL + RTOL * np.abs(ref)).all()
        assert h.get_error() == 0
    finally:
        h.destroy()
