"""GPU parity of the prefill attention against the CPU oracle, through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2401_05391_b200 import segkv as sk
from paper_2401_05391_b200 import workloads as wl

from _harness import ATOL, RTOL

pytestmark = pytest.mark.gpu


def check_rows(w, q, kp, vp, out, slopes, rows):
    ref = oracle.prefill_sdpa(w.dtype, w.batch, w.heads, w.kv_heads, w.head_dim, wl.to_bits(q), wl.to_bits(kp),
                              wl.to_bits(vp), slopes=None if slopes is None else slopes.cpu().numpy(), rows=rows)
    got = np.stack([out[b, i, h].to(torch.float64).cpu().numpy() for b, i, h in rows])
    assert np.isfinite(got).all()
    err = np.abs(got - ref)
    # the path's stated tolerance for both storage types
    assert (err <= ATOL + RTOL * np.abs(ref)).all(), f"max err {err.max():.3e}"


def run_prefill(w, rows_fn, row_groups=0, prompt_layout=None):
    h = sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype)
    try:
        h.set_prefill_tuning(row_groups)
        if prompt_layout is not None:
            h.set_prompt_layout(prompt_layout)
        kp, vp = wl.make_prompt(w, "cuda")
        q = wl.make_prefill_query(w, "cuda")
        slopes = wl.alibi_slopes(w.heads).cuda() if w.alibi else None
        out = torch.full_like(q, float("nan"))
        h.prefill(kp, vp, q, out, slopes)
        torch.cuda.synchronize()
        assert not torch.isnan(out.float()).any(), "unwritten outputs"
        check_rows(w, q, kp, vp, out, slopes, rows_fn(w))
        assert h.get_error() == 0
        return h, q, kp, vp, out, slopes
    except Exception:
        h.destroy()
        raise


def all_rows(w):
    return [(b, i, h) for b in range(w.batch) for i in range(w.prompt_len) for h in range(w.heads)]


def sampled_rows(w, n=192, seed=0):
    rng = np.random.default_rng(w.seed + seed)
    rows = {(0, 0, 0), (w.batch - 1, w.prompt_len - 1, w.heads - 1), (0, 63, 0), (0, 64, 0), (0, w.prompt_len - 1, 0)}
    while len(rows) < n:
        rows.add((int(rng.integers(w.batch)), int(rng.integers(w.prompt_len)), int(rng.integers(w.heads))))
    return sorted(r for r in rows if r[1] < w.prompt_len)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("D,P", [(64, 150), (128, 150), (128, 64), (128, 65), (64, 1), (256, 150), (256, 33), (128, 300)])
def test_prefill_ragged_small_shapes(dtype, D, P):
    # several tiles and a ragged tail, GQA, ALiBi on the bf16 variants
    w = wl.Workload("pf", 2, 3, 6, 2, D, P, 2, dtype, "uniform", dtype == "bf16", 80 + D // 64)
    h = run_prefill(w, all_rows)[0]
    h.destroy()


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("row_groups", [1, 2])
@pytest.mark.parametrize("P", [64, 128, 129, 150, 256, 257, 300, 520, 777])
def test_prefill_head_dim_128_row_groups(dtype, row_groups, P):
    # the tcgen05 kernel with one and with two 128-row groups per CTA: prompts that leave the
    # second group empty (64, 128), with one row (129), exact tiles (256), ragged (150, 257, 300, 777)
    # and spanning CTAs (520, 777)
    w = wl.Workload("pf", 2, 3, 4, 2, 128, P, 2, dtype, "uniform", dtype == "bf16", 90 + row_groups)
    h = run_prefill(w, all_rows if P <= 300 else (lambda w: sampled_rows(w, 400)), row_groups)[0]
    h.destroy()


@pytest.mark.parametrize("row_groups", [1, 2])
def test_prefill_llama2_7b_shape_row_groups_sampled(row_groups):
    h = run_prefill(wl.CONFIGS[1], lambda w: sampled_rows(w, 256), row_groups)[0]
    h.destroy()


@pytest.mark.parametrize("layout", ["token_major", "seq_first"])
@pytest.mark.parametrize("D,P", [(64, 150), (128, 300), (256, 150)])
def test_prefill_prompt_layouts(layout, D, P):
    w = wl.Workload("pf", 2, 3, 6, 2, D, P, 2, "f16", "uniform", False, 95)
    h = run_prefill(w, all_rows, prompt_layout=layout)[0]
    h.destroy()


@pytest.mark.parametrize("D,row_groups", [(256, 0), (128, 1), (64, 1), (64, 2)])
def test_prefill_many_items_per_cta(D, row_groups):
    # 768 or more work items on 148 persistent CTAs, tile counts 5 / 4 / 2 per item: every CTA walks
    # several items back to back (barrier phases, ring positions and tensor-memory buffers carry over)
    w = wl.Workload("pf", 16, 2, 16, 16, D, 300, 2, "f16", "uniform", False, 97)
    for _ in range(2):
        h = run_prefill(w, lambda w: sampled_rows(w, 300), row_groups)[0]
        h.destroy()


@pytest.mark.parametrize("dtype,D", [("f16", 128), ("bf16", 128), ("f16", 256), ("f16", 64)])
def test_prefill_per_request_prompt_lengths(dtype, D):
    # ragged prompts: each request is computed up to its own length (against the oracle run on that
    # request alone), the poisoned padding never leaks in, and the rows behind a request's length stay untouched
    lens = [300, 1, 129, 64, 257]
    w = wl.Workload("pf", len(lens), 2, 4, 2, D, 300, 2, dtype, "uniform", dtype == "bf16", 98)
    h = sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype)
    try:
        kp, vp = wl.make_prompt(w, "cuda")
        q = wl.make_prefill_query(w, "cuda")
        for b, n in enumerate(lens):
            kp[b, n:] = float("nan")
            vp[b, n:] = float("inf")
        slopes = wl.alibi_slopes(w.heads).cuda() if w.alibi else None
        for groups in (1, 2):
            if D == 256 and groups == 2:
                continue
            h.set_prefill_tuning(groups)
            h.prefill_write_ragged(kp, vp, lens)
            out = torch.full_like(q, 512.0)
            h.prefill_sdpa(q, out, slopes)
            torch.cuda.synchronize()
            assert h.get_error() == 0
            for b, n in enumerate(lens):
                assert bool((out[b, n:].float() == 512.0).all()), "rows behind the request's length were written"
                w1 = w.scaled(batch=1, prompt_len=n)
                rows = [(0, i, hd) for i in sorted({0, n - 1, n // 2, min(n - 1, 63), min(n - 1, 128)}) for hd in range(w.heads)]
                check_rows(w1, q[b:b + 1, :n].contiguous(), kp[b:b + 1, :n].contiguous(), vp[b:b + 1, :n].contiguous(),
                           out[b:b + 1, :n].contiguous(), slopes, rows)
    finally:
        h.destroy()


@pytest.mark.parametrize("layout", [None, "token_major", "seq_first"])
@pytest.mark.parametrize("dtype,D,heads,kv_heads,P", [("f16", 128, 8, 2, 300), ("bf16", 128, 4, 4, 129), ("f16", 256, 4, 2, 150),
                                                      ("f16", 64, 6, 3, 520)])
def test_fused_prefill_stores_the_same_segment_and_output_as_the_two_calls(layout, dtype, D, heads, kv_heads, P):
    # segkv_prefill (one launch: attention + prompt store) against segkv_prefill_write + segkv_prefill_sdpa:
    # same output bit for bit, and the decode attention over the stored segment agrees bit for bit too
    w = wl.Workload("pf", 3, 2, heads, kv_heads, D, P, 3, dtype, "uniform", dtype == "bf16", 99)
    kp, vp = wl.make_prompt(w, "cuda")
    q = wl.make_prefill_query(w, "cuda")
    slopes = wl.alibi_slopes(w.heads).cuda() if w.alibi else None
    qd, kd, vd = wl.make_step(w, 0, "cuda")
    results = []
    for fused in (False, True):
        h = sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len + 40, w.steps, w.torch_dtype)
        try:
            if layout is not None:
                h.set_prompt_layout(layout)
            out = torch.full_like(q, 512.0)
            if fused:
                h.prefill(kp, vp, q, out, slopes)
            else:
                h.prefill_write(kp, vp)
                h.prefill_sdpa(q, out, slopes)
            dec0 = h.decode_sdpa(qd, None, slopes)                 # prompt only
            h.append(0, None, kd, vd)
            dec1 = h.decode_sdpa(qd, None, slopes)
            torch.cuda.synchronize()
            assert h.get_error() == 0
            results.append((out.clone(), dec0.clone(), dec1.clone()))
        finally:
            h.destroy()
    for a, b in zip(*results):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    check_rows(w, q, kp, vp, results[1][0], slopes, sampled_rows(w, 96))


@pytest.mark.parametrize("D,H,Hkv,P,groups", [(256, 16, 16, 300, 0), (128, 16, 4, 300, 1), (128, 16, 16, 520, 2)])
def test_prefill_is_bit_reproducible_across_runs(D, H, Hkv, P, groups):
    # no atomics and a fixed schedule: repeated launches must give the same bits (a missed barrier phase
    # once showed up here as rows that changed from run to run)
    w = wl.Workload("pf", 16, 2, H, Hkv, D, P, 2, "f16", "uniform", False, 96)
    h = sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype)
    try:
        h.set_prefill_tuning(groups)
        kp, vp = wl.make_prompt(w, "cuda")
        q = wl.make_prefill_query(w, "cuda")
        ref = None
        for it in range(10):
            out = torch.full_like(q, 512.0)
            if it % 2:
                h.prefill(kp, vp, q, out)
            else:
                h.prefill_write(kp, vp)
                h.prefill_sdpa(q, out)
            torch.cuda.synchronize()
            assert not torch.isnan(out.float()).any()
            if ref is None:
                ref = out.clone()
            assert torch.equal(ref.view(torch.int16), out.view(torch.int16)), f"run {it} differs"
        assert h.get_error() == 0
    finally:
        h.destroy()


@pytest.mark.parametrize("D,H,Hkv,P", [(128, 8, 8, 4096), (256, 8, 2, 3000)])
def test_prefill_long_prompt_sampled(D, H, Hkv, P):
    # 32 or more key tiles per row group, items of very different lengths on every CTA
    w = wl.Workload("pf", 1, 2, H, Hkv, D, P, 2, "f16", "uniform", False, 94)
    h = run_prefill(w, lambda w: sampled_rows(w, 96))[0]
    h.destroy()


def test_prefill_llama2_7b_shape_sampled():
    h = run_prefill(wl.CONFIGS[1], lambda w: sampled_rows(w, 256))[0]
    h.destroy()


def test_prefill_gptj_shape_cut_to_batch_2_sampled():
    h = run_prefill(wl.CONFIGS[2].scaled(batch=2), lambda w: sampled_rows(w, 256))[0]
    h.destroy()


def test_prefill_bloom_shape_cut_to_batch_2_sampled():
    h = run_prefill(wl.CONFIGS[4].scaled(batch=2), lambda w: sampled_rows(w, 256))[0]
    h.destroy()


def test_prefill_last_row_agrees_with_the_decode_kernel_on_the_prompt():
    """The prefill kernel is the decode kernel's special case: its last row is what the decode
    kernel returns for a query that sees only the prompt."""
    w = wl.Workload("pfdec", 2, 4, 4, 2, 128, 200, 2, "f16", "uniform", True, 83)
    h, q, kp, vp, out, slopes = run_prefill(w, lambda w: sampled_rows(w, 64))
    try:
        qd = q[:, -1].repeat_interleave(w.beams, dim=0).contiguous()        # [rows, heads, D]
        od = h.decode_sdpa(qd, None, slopes)
        torch.cuda.synchronize()
        want = out[:, -1].repeat_interleave(w.beams, dim=0)
        assert torch.allclose(od.float(), want.float(), atol=2e-3, rtol=1e-2)
    finally:
        h.destroy()


def test_prefill_argument_and_state_errors():
    h = sk.SegKV(1, 2, 2, 2, 64, 16, 4, torch.float16)
    q = torch.zeros(1, 16, 2, 64, dtype=torch.float16, device="cuda")
    with pytest.raises(sk.SegKVError) as e:
        rc = sk.lib().segkv_prefill_sdpa(h._h, q.data_ptr(), q.data_ptr(), None, None)
        sk._check(rc, "segkv_prefill_sdpa")
    assert e.value.code == sk.SEGKV_ESTATE                   # no prompt stored yet
    rc = sk.lib().segkv_prefill_sdpa(h._h, None, q.data_ptr(), None, None)
    assert rc == sk.SEGKV_EINVAL
    h.destroy()
