"""GPU parity: the CUDA path against the CPU oracle, element by element, through the C-ABI."""
import numpy as np
import pytest
import torch

from paper_2401_05391_b200 import workloads as wl
from paper_2401_05391_b200 import segkv as sk

from _harness import Run, all_pairs, sampled_pairs, unique_rows_from_ancestry

pytestmark = pytest.mark.gpu

CHECK_STEPS = (0, 1, 2, 3, 7, 15, 16, 17, 31, 63, 127, 255)


def run_workload(w, pairs_fn, check_steps=CHECK_STEPS, splits=0, stages=0, combine=0, every_step_ancestry=True,
                 prompt_layout=None, prompt_lens=None, tile=0, persistent=-1, chunk_steps=0):
    r = Run(w, splits=splits, stages=stages, combine=combine, prompt_layout=prompt_layout, prompt_lens=prompt_lens,
            tile=tile, persistent=persistent, chunk_steps=chunk_steps)
    try:
        worst = 0.0
        for t in range(w.steps):
            r.append_next()
            if every_step_ancestry or t in check_steps or t == w.steps - 1:
                anc = r.h.get_ancestry()
                ref = r.oracle_ancestry(t)
                assert np.array_equal(anc, ref), f"beam-index table differs at step {t}"
                assert np.array_equal(r.h.get_unique_rows(), unique_rows_from_ancestry(ref, w.batch, w.beams))
            if t in check_steps or t == w.steps - 1:
                out, q = r.decode()
                worst = max(worst, r.check(out, q, t, pairs_fn(w)))
        assert r.h.get_error() == 0
        return worst
    finally:
        r.close()


def run_workload_fused(w, pairs_fn, check_steps=CHECK_STEPS, splits=0, stages=0, combine=0, prompt_layout=None,
                       prompt_lens=None, tile=0):
    """Same as run_workload but every step is one fused segkv_decode_step launch."""
    r = Run(w, splits=splits, stages=stages, combine=combine, prompt_layout=prompt_layout, prompt_lens=prompt_lens,
            tile=tile)
    try:
        for t in range(w.steps):
            _, out, q = r.step_fused()
            if t in check_steps or t == w.steps - 1:
                ref = r.oracle_ancestry(t)
                assert np.array_equal(r.h.get_ancestry(), ref), f"beam-index table differs at step {t}"
                assert np.array_equal(r.h.get_unique_rows(), unique_rows_from_ancestry(ref, w.batch, w.beams))
                r.check(out, q, t, pairs_fn(w))
        assert r.h.get_error() == 0
    finally:
        r.close()


def test_fused_step_tiny_every_step():
    w = wl.CONFIGS[0]
    run_workload_fused(w, all_pairs, check_steps=tuple(range(w.steps)))


def test_fused_step_llama2_7b_shape():
    run_workload_fused(wl.CONFIGS[1], all_pairs)


@pytest.mark.parametrize("idx", [2, 3, 4])
def test_fused_step_large_shapes_sampled(idx):
    run_workload_fused(wl.CONFIGS[idx], lambda w: sampled_pairs(w, 24), check_steps=(0, 1, 17, 127, 255))


@pytest.mark.parametrize("dtype,D,splits,combine", [("f16", 64, 4, 1), ("bf16", 128, 4, 2), ("f16", 256, 4, 1),
                                                    ("f16", 128, 1, 0), ("bf16", 64, 7, 0)])
def test_fused_step_ragged_shapes(dtype, D, splits, combine):
    # a forced single split still runs the fused kernel (several response tiles per CTA)
    w = wl.Workload("ragged-fused", 3, 3, 6, 2, D, 150, 40, dtype, "uniform", dtype == "bf16", 60 + D // 64)
    run_workload_fused(w, all_pairs, check_steps=(0, 1, 5, 20, 39), splits=splits, combine=combine)


def test_fused_step_long_response_single_split():
    # 200 steps x 4 beams through one CTA per work group: windows, tile spill-over, ring reuse
    w = wl.Workload("long-fused", 2, 4, 2, 2, 128, 100, 200, "f16", "half_identity", False, 66)
    run_workload_fused(w, all_pairs, check_steps=(0, 15, 16, 17, 63, 64, 65, 130, 199), splits=1)


def test_fused_and_separate_calls_mix():
    """A fused step leaves the cache, parents and table exactly as append would: later separate
    calls (and the other way round) continue from it."""
    w = wl.CONFIGS[0].scaled(steps=12, prompt_len=70, index=61)
    r = Run(w)
    try:
        for t in range(w.steps):
            if t % 3 == 0:
                r.append_next()
                out, q = r.decode()
            else:
                _, out, q = r.step_fused()
                again, _ = r.decode(q)                     # the separate kernel on the state the fused step left
                # same result up to the order in which keys are summed (the two forms cut the
                # response rows into tiles differently)
                assert torch.allclose(out.float(), again.float(), atol=2e-3, rtol=1e-2)
            assert np.array_equal(r.h.get_ancestry(), r.oracle_ancestry(t))
            r.check(out, q, t, all_pairs(w))
        # re-time a fused step: drop it, run it again, same bits
        r.h.truncate_last()
        t = w.steps - 1
        out2 = r.h.decode_step(t, r.parents_dev[t], r.k_steps[t], r.v_steps[t], q, None, r.slopes)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), out2.view(torch.int16))
    finally:
        r.close()


def test_fused_step_wide_beam_and_single_beam():
    run_workload_fused(wl.Workload("w1f", 2, 1, 4, 4, 128, 77, 9, "f16", "uniform", False, 62), all_pairs)
    run_workload_fused(wl.Workload("w8f", 2, 8, 2, 2, 64, 77, 40, "f16", "uniform", False, 63), all_pairs,
                       check_steps=(0, 3, 39))
    run_workload_fused(wl.Workload("w16f", 1, 16, 2, 2, 64, 40, 24, "f16", "uniform", False, 64), all_pairs,
                       check_steps=(0, 3, 23))


@pytest.mark.parametrize("fused", [False, True])
def test_growing_capacity_matches_fixed_capacity_and_eq3(fused):
    """Response capacity in 16-step chunks (the paper's N_step policy): same bits as the fixed-capacity
    cache at every step, and the K/V bytes held follow Eq. 3."""
    import oracle
    w = wl.Workload("grow", 2, 4, 4, 2, 128, 96, 50, "f16", "uniform", False, 67)
    a, b = Run(w), Run(w, chunk_steps=16)
    try:
        tok = oracle.cache_token(1, w.kv_heads, w.head_dim, 2)
        for t in range(w.steps):
            if fused:
                _, oa, q = a.step_fused()
                _, ob, _ = b.step_fused()
            else:
                a.append_next(); b.append_next()
                oa, q = a.decode()
                ob, _ = b.decode(q)
            assert torch.equal(oa.view(torch.int16), ob.view(torch.int16)), f"step {t}"
            assert b.h.allocated_kv_bytes == oracle.cache_segment(w.batch, w.beams, w.prompt_len, t + 1, tok, 16)
            assert a.h.allocated_kv_bytes == sk.segkv_storage_bytes(w.batch, w.beams, w.kv_heads, w.head_dim,
                                                                   w.prompt_len, w.steps, sk.SEGKV_F16)
        assert np.array_equal(a.h.get_ancestry(), b.h.get_ancestry())
        b.check(ob, q, w.steps - 1, all_pairs(w))
        x = b.h.decode_sdpa_rowwise(q, None, None)           # the per-beam kernel walks the chunks too
        torch.cuda.synchronize()
        assert torch.allclose(x.float(), ob.float(), atol=4e-3, rtol=2e-2)
        assert a.h.get_error() == 0 and b.h.get_error() == 0
    finally:
        a.close(); b.close()


def test_tiny_every_step_all_outputs():
    w = wl.CONFIGS[0]
    run_workload(w, all_pairs, check_steps=tuple(range(w.steps)))


def test_llama2_7b_shape():
    run_workload(wl.CONFIGS[1], all_pairs)


def test_gptj_shape_sampled():
    run_workload(wl.CONFIGS[2], lambda w: sampled_pairs(w, 64), every_step_ancestry=False)


@pytest.mark.parametrize("idx", [3, 4])
def test_large_shapes_sampled(idx):
    w = wl.CONFIGS[idx]
    run_workload(w, lambda w: sampled_pairs(w, 64), check_steps=(0, 17, 127, 255), every_step_ancestry=False)


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("D", [64, 128, 256])
def test_ragged_small_shapes(dtype, D):
    # prompt not a multiple of the tile, several tiles, GQA, ALiBi on one variant
    w = wl.Workload("ragged", 3, 3, 6, 2, D, 150, 21, dtype, "uniform", dtype == "bf16", 10 + D // 64)
    run_workload(w, all_pairs, check_steps=(0, 1, 5, 20))


@pytest.mark.parametrize("splits,stages,combine", [(1, 0, 0), (2, 2, 1), (2, 2, 2), (4, 0, 2), (5, 1, 0), (8, 3, 1),
                                                   (8, 0, 2), (19, 3, 0), (40, 0, 0)])
def test_forced_splits_stages_and_combine(splits, stages, combine):
    # more splits than tiles leaves some CTAs without keys; one stage serialises the ring;
    # combine 1 = workspace + ticket, 2 = thread-block cluster
    w = wl.CONFIGS[1].scaled(steps=40, index=30)
    run_workload(w, lambda w: sampled_pairs(w, 12), check_steps=(0, 7, 39), splits=splits, stages=stages,
                 combine=combine, every_step_ancestry=False)


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("splits,stages,combine", [(0, 0, 0), (1, 0, 0), (8, 0, 1), (8, 0, 2), (16, 2, 1), (5, 1, 0), (4, 3, 2)])
def test_small_cta_form_forced_shapes(splits, stages, combine, fused):
    # the 32-key-tile form of the kernel (two consumer warps, quarter-SM CTAs) in every merge mode
    w = wl.CONFIGS[1].scaled(steps=40, index=31)
    run = run_workload_fused if fused else run_workload
    kw = {} if fused else {"every_step_ancestry": False}
    run(w, lambda w: sampled_pairs(w, 12), check_steps=(0, 7, 39), splits=splits, stages=stages, combine=combine,
        tile=32, **kw)


@pytest.mark.parametrize("splits", [0, 1, 2, 3, 5, 8])
def test_persistent_form_llama2_7b_shape(splits):
    # resident CTAs walking (work group, split) items round-robin; 1 to 8 items per work group
    w = wl.CONFIGS[1].scaled(steps=40, index=33)
    run_workload(w, lambda w: sampled_pairs(w, 12), check_steps=(0, 7, 39), splits=splits, persistent=1,
                 every_step_ancestry=False)


@pytest.mark.parametrize("dtype,D", [("f16", 64), ("bf16", 128), ("f16", 256)])
def test_persistent_form_ragged_shapes(dtype, D):
    # prompt not a multiple of the tile, GQA (6 query columns), ALiBi on the bf16 variant, per-request
    # prompt lengths, a response capacity that grows in chunks, more items than resident CTAs
    w = wl.Workload("pers", 3, 3, 6, 3, D, 150, 21, dtype, "uniform", dtype == "bf16", 70 + D // 64)
    run_workload(w, all_pairs, check_steps=(0, 1, 5, 20), persistent=1)
    run_workload(w, all_pairs, check_steps=(0, 5, 20), persistent=1, splits=2, prompt_lens=[150, 33, 97])
    run_workload(w, all_pairs, check_steps=(0, 5, 20), persistent=1, splits=3, chunk_steps=4)
    big = wl.Workload("pers_many", 40, 2, 16, 16, D, 70, 5, dtype, "uniform", dtype == "bf16", 80 + D // 64)
    run_workload(big, lambda w: sampled_pairs(w, 40), check_steps=(0, 4), persistent=1)
    run_workload(big, lambda w: sampled_pairs(w, 40), check_steps=(0, 4), persistent=1, splits=2)


@pytest.mark.parametrize("dtype,D,hkv", [("f16", 128, 16), ("bf16", 64, 16), ("f16", 256, 8)])
def test_ragged_last_wave_is_cut_finer(dtype, D, hkv):
    # more work groups than CTA slots with a short last wave (640 or 320 on 296 slots): the groups of that
    # wave are cut into splits and merged through the workspace, the others store their output directly
    w = wl.Workload("tail", 40, 2, hkv, hkv, D, 300, 5, dtype, "uniform", dtype == "bf16", 95 + D // 64)
    pairs = sorted(set(sampled_pairs(w, 24)) | {(b, h) for b in (36, 37, 38, 39) for h in (0, 3, hkv - 1)})
    run_workload(w, lambda w: pairs, check_steps=(0, 4), every_step_ancestry=False)
    run_workload(w, lambda w: pairs, check_steps=(0, 4), every_step_ancestry=False, prompt_lens=[300 - 7 * (b % 5) for b in range(40)])


def test_persistent_form_no_prompt_and_first_step():
    # no prompt at all (only response rows), and a prompt with no step yet (an empty response tile)
    w = wl.Workload("pers_np", 2, 4, 4, 4, 128, 0, 12, "f16", "uniform", False, 91)
    run_workload(w, all_pairs, check_steps=(0, 3, 11), persistent=1)
    w = wl.Workload("pers_ponly", 2, 4, 4, 4, 128, 100, 4, "f16", "uniform", False, 92)
    r = Run(w, persistent=1)
    try:
        out, q = r.decode()
        r.check(out, q, -1, all_pairs(w))
    finally:
        r.close()


@pytest.mark.parametrize("dtype,D", [("f16", 64), ("bf16", 128)])
def test_small_cta_form_ragged_shapes(dtype, D):
    # prompt not a multiple of the 32-key tile, GQA (6 query columns), ALiBi on the bf16 variant, ragged lengths
    w = wl.Workload("ragged32", 3, 3, 6, 3, D, 150, 21, dtype, "uniform", dtype == "bf16", 14 + D // 64)
    run_workload(w, all_pairs, check_steps=(0, 1, 5, 20), tile=32)
    run_workload_fused(w, all_pairs, check_steps=(0, 1, 5, 20), tile=32, splits=3)
    run_workload(w, all_pairs, check_steps=(0, 5, 20), tile=32, prompt_lens=[150, 33, 97])


def test_cluster_combine_small_shapes():
    for D, dt in ((64, "f16"), (256, "bf16")):
        w = wl.Workload("cl", 2, 3, 4, 2, D, 300, 9, dt, "uniform", True, 40 + D)
        run_workload(w, all_pairs, check_steps=(0, 8), splits=4, combine=2)


@pytest.mark.parametrize("layout", ["token_major", "seq_first"])
@pytest.mark.parametrize("dtype,D", [("f16", 64), ("bf16", 128), ("f16", 256)])
def test_prompt_layouts_ragged_shapes(layout, dtype, D):
    # the prompt segment kept token-major ([B, P, Hkv, D], the paper's) or sequence-first instead of
    # head-major: separate calls and the fused step, GQA, ragged prompt, ALiBi on the bf16 variant
    w = wl.Workload("layout", 3, 3, 6, 2, D, 150, 9, dtype, "uniform", dtype == "bf16", 60 + D // 64)
    run_workload(w, all_pairs, check_steps=(0, 8), prompt_layout=layout)
    run_workload_fused(w, all_pairs, check_steps=(0, 8), splits=3, prompt_layout=layout)


@pytest.mark.parametrize("layout", ["token_major", "seq_first"])
def test_prompt_layouts_llama2_7b_shape_and_rowwise(layout):
    w = wl.CONFIGS[1]
    r = Run(w, prompt_layout=layout)
    try:
        r.advance_to(w.steps - 1)
        out, q = r.decode()
        r.check(out, q, w.steps - 1, sampled_pairs(w, 64))
        b = r.h.decode_sdpa_rowwise(q, None, r.slopes)
        torch.cuda.synchronize()
        r.check(b, q, w.steps - 1, sampled_pairs(w, 64))
        assert r.h.get_error() == 0
    finally:
        r.close()


def test_prompt_layout_can_only_change_while_no_prompt_is_stored():
    w = wl.CONFIGS[0]
    r = Run(w)
    try:
        with pytest.raises(sk.SegKVError):
            r.h.set_prompt_layout("token_major")
        with pytest.raises(sk.SegKVError):
            r.h.set_prompt_layout(7)
        r.h.reset(keep_prompt=False)
        r.h.set_prompt_layout("token_major")
        r.h.prefill_write(r.kp, r.vp)
        r.advance_to(2)
        out, q = r.decode()
        r.check(out, q, 2, all_pairs(w))
    finally:
        r.close()


@pytest.mark.parametrize("dtype,D,layout", [("f16", 64, None), ("bf16", 128, None), ("f16", 256, None),
                                            ("bf16", 128, "token_major")])
def test_per_request_prompt_lengths(dtype, D, layout):
    # every request with its own prompt length (1, a full tile, ragged, the padded length), NaN / inf in
    # the padding, ALiBi positions counted from each request's own length on the bf16 variants
    w = wl.Workload("plens", 5, 3, 6, 2, D, 200, 9, dtype, "uniform", dtype == "bf16", 70 + D // 64)
    lens = [1, 64, 150, 200, 65]
    for splits in (0, 3):
        run_workload(w, all_pairs, check_steps=(0, 8), splits=splits, prompt_layout=layout, prompt_lens=lens)
        run_workload_fused(w, all_pairs, check_steps=(0, 8), splits=splits, prompt_layout=layout, prompt_lens=lens)


def test_per_request_prompt_lengths_rowwise_and_errors():
    w = wl.Workload("plens", 3, 4, 4, 4, 128, 100, 5, "f16", "uniform", True, 77)
    r = Run(w, prompt_lens=[100, 3, 37])
    try:
        r.advance_to(4)
        out, q = r.decode()
        r.check(out, q, 4, all_pairs(w))
        b = r.h.decode_sdpa_rowwise(q, None, r.slopes)
        torch.cuda.synchronize()
        r.check(b, q, 4, all_pairs(w))
        for bad in ([100, 0, 37], [100, 101, 37]):
            with pytest.raises(sk.SegKVError):
                r.h.prefill_write_ragged(r.kp, r.vp, bad)
        # back to one length for all: the padding written above is what the requests now see
        clean_k, clean_v = wl.make_prompt(w, "cuda")
        r.kp, r.vp, r.prompt_lens = clean_k, clean_v, None
        r.h.prefill_write(clean_k, clean_v)
        r.k_steps, r.v_steps, r.q_steps = [], [], []
        r.advance_to(1)
        out, q = r.decode()
        r.check(out, q, 1, all_pairs(w))
    finally:
        r.close()


@pytest.mark.parametrize("style", ["half", "interleaved"])
@pytest.mark.parametrize("dtype,D,ragged", [("f16", 64, False), ("bf16", 128, True), ("f16", 256, False)])
def test_append_with_rotary_embedding(style, dtype, D, ragged):
    # K rows rotated on their way into the response segment: the attention over them must match the
    # oracle fed with K rows rotated by the oracle's own embedding (GQA, per-request positions when ragged)
    w = wl.Workload("rope", 3, 3, 6, 2, D, 90, 7, dtype, "uniform", False, 80 + D // 64)
    lens = [90, 17, 64] if ragged else None
    cos, sin = [t.cuda() for t in wl.rope_tables(128, D)]
    r = Run(w, prompt_lens=lens)
    try:
        for t in range(w.steps):
            r.append_next_rope(cos, sin, style)
            if t in (0, 3, w.steps - 1):
                out, q = r.decode()
                r.check(out, q, t, all_pairs(w))
        assert r.h.get_error() == 0
        assert np.array_equal(r.h.get_ancestry(), r.oracle_ancestry(w.steps - 1))
    finally:
        r.close()


def test_append_with_rotary_embedding_errors():
    w = wl.CONFIGS[0]
    cos, sin = [t.cuda() for t in wl.rope_tables(w.prompt_len + 2, w.head_dim)]
    r = Run(w)
    try:
        q, k, v = wl.make_step(w, 0, "cuda")
        with pytest.raises(sk.SegKVError):
            r.h.append_rope(0, None, k, v, cos, sin, 3)                 # unknown style
        r.h.append_rope(0, None, k, v, cos, sin, "half")
        r.h.append_rope(1, r.parents_dev[1], k, v, cos, sin, "half")
        with pytest.raises(sk.SegKVError):
            r.h.append_rope(2, r.parents_dev[2], k, v, cos, sin, "half")   # position prompt_len + 2 is past the tables
        assert r.h.steps == 2
    finally:
        r.close()


@pytest.mark.parametrize("leader_fused", [False, True])
def test_layers_share_one_beam_index_table(leader_fused):
    # three "layers" with their own K/V and one set of tables: the leader updates them (by the separate
    # append or inside the fused step), the followers store rows only and attend through the leader's tables
    base = wl.Workload("share", 2, 4, 8, 4, 128, 130, 12, "f16", "uniform", False, 90)
    layers = [Run(base.scaled(index=90 + 7 * i), parents=wl.make_parents(base), splits=4) for i in range(3)]
    lead, followers = layers[0], layers[1:]
    try:
        for f in followers:
            f.h.share_index(lead.h)
        with pytest.raises(sk.SegKVError):
            lead.h.share_index(followers[0].h)                     # a leader cannot follow its follower
        q0, k0, v0 = wl.make_step(followers[0].w, 0, "cuda")
        with pytest.raises(sk.SegKVError):
            followers[0].h.append(0, None, k0, v0)                 # the leader has not made step 0 yet
        for t in range(base.steps):
            if leader_fused:
                _, out, q = lead.step_fused()
            else:
                lead.append_next()
                out, q = lead.decode()
            if t in (0, 5, base.steps - 1):
                lead.check(out, q, t, all_pairs(base))
            for f in followers:
                if t % 2:
                    _, out, q = f.step_fused()                     # runs as append + attention on a follower
                else:
                    f.append_next()
                    out, q = f.decode()
                if t in (0, 5, base.steps - 1):
                    f.check(out, q, t, all_pairs(base))
                    assert np.array_equal(f.h.get_ancestry(), lead.oracle_ancestry(t))
        for r in layers:
            assert r.h.get_error() == 0
        assert sk.lib().segkv_destroy(lead.h._h) == -2           # ESTATE: two handles still follow it
        followers[0].h.reset()
        followers[0].h.share_index(None)
        with pytest.raises(sk.SegKVError):
            followers[1].h.share_index(None)                       # not at step 0
    finally:
        for r in reversed(layers):
            r.close()


def test_tiled_kernel_agrees_with_rowwise_kernel():
    w = wl.Workload("cross", 2, 4, 8, 4, 128, 333, 30, "bf16", "uniform", True, 31)
    r = Run(w)
    try:
        r.advance_to(29)
        a, q = r.decode()
        b = r.h.decode_sdpa_rowwise(q, None, r.slopes)
        torch.cuda.synchronize()
        assert torch.allclose(a.float(), b.float(), atol=4e-3, rtol=2e-2)
    finally:
        r.close()


def test_prompt_only_and_response_only():
    w = wl.Workload("ponly", 2, 4, 4, 4, 128, 100, 4, "f16", "uniform", False, 20)
    r = Run(w)
    try:
        out, q = r.decode()
        r.check(out, q, -1, all_pairs(w))
    finally:
        r.close()
    w0 = w.scaled(prompt_len=0, index=21, steps=70)
    run_workload(w0, all_pairs, check_steps=(0, 1, 33, 69))


def test_single_beam_and_wide_beam():
    run_workload(wl.Workload("w1", 2, 1, 4, 4, 128, 77, 9, "f16", "uniform", False, 22), all_pairs)
    run_workload(wl.Workload("w8", 2, 8, 2, 2, 64, 77, 40, "f16", "uniform", False, 23), all_pairs,
                 check_steps=(0, 3, 39))


def test_sixteen_query_columns_and_the_rowwise_fallback():
    # 16 columns per kv head (two column tiles) is the most the tiled kernel takes ...
    run_workload(wl.Workload("c16", 2, 4, 8, 2, 128, 130, 20, "f16", "uniform", True, 24), all_pairs,
                 check_steps=(0, 7, 19))
    run_workload(wl.Workload("c16b", 1, 16, 2, 2, 64, 70, 20, "bf16", "uniform", False, 25), all_pairs,
                 check_steps=(0, 19))
    # ... beyond that (here 32 beams) the per-beam kernel serves segkv_decode_sdpa and segkv_decode_step
    w = wl.Workload("w32", 1, 32, 2, 2, 64, 40, 12, "f16", "uniform", False, 26)
    run_workload(w, all_pairs, check_steps=(0, 5, 11))
    run_workload_fused(w, all_pairs, check_steps=(0, 5, 11))


@pytest.mark.parametrize("kind", ["identity", "collapse", "cycle"])
def test_degenerate_parent_tables(kind):
    """identity: beams never mix (every response row is read by one beam); collapse: every beam
    extends beam 0 (one shared row per step); cycle: the beams rotate."""
    w = wl.Workload("deg-" + kind, 2, 4, 4, 4, 128, 90, 33, "f16", "uniform", False, 27)
    j = np.tile(np.arange(w.beams), w.batch)
    row = {"identity": j, "collapse": np.zeros_like(j), "cycle": (j + 1) % w.beams}[kind]
    par = np.tile(row, (w.steps, 1)).astype(np.int32)
    for fused in (False, True):
        r = Run(w, parents=par)
        try:
            for t in range(w.steps):
                if fused:
                    _, out, q = r.step_fused()
                else:
                    r.append_next()
            if not fused:
                out, q = r.decode()
            t = w.steps - 1
            assert np.array_equal(r.h.get_ancestry(), r.oracle_ancestry(t))
            uniq = r.h.get_unique_rows()
            if kind == "identity" or kind == "cycle":
                assert (uniq == w.beams * w.steps).all()
            else:
                assert (uniq == w.steps + w.beams - 1).all()       # one row per step, W at the newest
            r.check(out, q, t, all_pairs(w))
        finally:
            r.close()


def test_one_key_only():
    # a single prompt key and no response: the output is that key's value row, for every beam
    w = wl.Workload("one", 2, 4, 2, 2, 128, 1, 1, "f16", "uniform", False, 28)
    r = Run(w)
    try:
        out, q = r.decode()
        want = r.vp[:, 0].repeat_interleave(w.beams, dim=0)        # [rows, kv_heads, D]
        assert torch.equal(out.view(torch.int16), want.view(torch.int16))
    finally:
        r.close()


def test_repeat_is_bit_identical_and_every_output_is_written():
    w = wl.CONFIGS[1].scaled(steps=24)
    r = Run(w)
    try:
        r.advance_to(23)
        a, q = r.decode()
        b, _ = r.decode(q)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        assert not torch.isnan(a.float()).any()
    finally:
        r.close()


def test_truncate_and_reappend_gives_same_result():
    w = wl.CONFIGS[0]
    r = Run(w)
    try:
        r.advance_to(5)
        a, q = r.decode()
        anc = r.h.get_ancestry()
        r.h.truncate_last()
        with pytest.raises(sk.SegKVError):
            r.h.truncate_last()
        r.h.append(5, r.parents_dev[5], r.k_steps[5], r.v_steps[5])
        b, _ = r.decode(q)
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        assert np.array_equal(anc, r.h.get_ancestry())
    finally:
        r.close()


def test_step_host_matches_device_calls():
    w = wl.CONFIGS[0]
    r = Run(w)
    r2 = Run(w)
    try:
        for t in range(w.steps):
            r.append_next()
            out, q = r.decode()
            qh, kh, vh = (x.cpu().pin_memory() for x in (q, r.k_steps[t], r.v_steps[t]))
            oh = torch.empty_like(qh).pin_memory()
            ph = torch.from_numpy(r.parents[t]).pin_memory() if t > 0 else None
            r2.h.step_host(t, ph, kh, vh, qh, oh)
            # the host step runs as one fused launch at this size, the device calls as two: the same rows in a
            # different order, so the two agree within the path's tolerance, not bit by bit
            assert torch.allclose(oh.float(), out.cpu().float(), atol=2e-3, rtol=1e-2)
            r.check(oh.to("cuda"), q, t, all_pairs(w))
    finally:
        r.close(); r2.close()


def test_step_host_packed_matches_device_calls():
    # one packed host block in, one copy out: same bits as the device-pointer calls (ALiBi slopes in the block too)
    w = wl.Workload("packed", 2, 4, 8, 4, 128, 150, 6, "bf16", "uniform", True, 123)
    r = Run(w)
    r2 = Run(w)
    try:
        total, off = r2.h.host_pack_layout()
        assert all(o % 256 == 0 for o in off) and total > off[4]
        blk = torch.zeros(total, dtype=torch.uint8).pin_memory()
        oh = torch.empty((w.rows, w.heads, w.head_dim), dtype=w.torch_dtype).pin_memory()

        def put(o, t):
            raw = t.contiguous().cpu().view(torch.uint8).reshape(-1)
            blk[o:o + raw.numel()] = raw
        put(off[1], r.slopes)
        for t in range(w.steps):
            r.append_next()
            out, q = r.decode()
            if t > 0:
                put(off[0], torch.from_numpy(r.parents[t]))
            put(off[2], r.k_steps[t]); put(off[3], r.v_steps[t]); put(off[4], q)
            if t % 2:
                r2.h.step_host_packed(t, blk, oh, has_slopes=True)
            else:                                            # queued only: the caller waits
                r2.h.step_host_packed_async(t, blk, oh, has_slopes=True)
                torch.cuda.synchronize()
            assert torch.allclose(oh.float(), out.cpu().float(), atol=4e-3, rtol=2e-2)
        assert np.array_equal(r2.h.get_ancestry(), r.h.get_ancestry())
        assert r2.h.get_error() == 0
    finally:
        r.close(); r2.close()


@pytest.mark.parametrize("one_array,heads,layers", [(False, 8, 3), (True, 8, 3), (True, 32, 6)])
def test_layers_step_host_queues_every_layer_in_one_call(one_array, heads, layers):
    # layers driven from pinned host blocks with one call per step; redo re-times the newest step.  Blocks
    # that are slices of one pinned array travel several layers per copy (32 heads, 6 layers: two groups).
    w = wl.Workload("stack", 1, 4, heads, heads, 128, 300, 6, "bf16", "uniform", True, 120)
    par = wl.make_parents(w)
    ls = [Run(w.scaled(index=120 + i), parents=par) for i in range(layers)]
    hs = [sk.SegKV(w.batch, w.beams, w.heads, w.kv_heads, w.head_dim, w.prompt_len, w.steps, w.torch_dtype) for _ in ls]
    try:
        total, off = hs[0].host_pack_layout()
        if one_array:
            blk_all = torch.zeros(layers, total, dtype=torch.uint8).pin_memory()
            out_all = torch.empty(layers, w.rows, w.heads, w.head_dim, dtype=w.torch_dtype).pin_memory()
            blks = [blk_all[i] for i in range(layers)]
            outs = [out_all[i] for i in range(layers)]
        else:
            blks = [torch.zeros(total, dtype=torch.uint8).pin_memory() for _ in ls]
            outs = [torch.empty(w.rows, w.heads, w.head_dim, dtype=w.torch_dtype).pin_memory() for _ in ls]
        for r, h in zip(ls, hs):
            h.prefill_write(r.kp, r.vp)
        stack = sk.LayerStack(hs, blks, outs)
        for t in range(w.steps):
            refs = []
            for r, blk in zip(ls, blks):
                r.append_next()
                out, q = r.decode()
                refs.append(out)

                def put(o, x):
                    raw = x.contiguous().cpu().view(torch.uint8).reshape(-1)
                    blk[o:o + raw.numel()] = raw
                if t > 0:
                    put(off[0], torch.from_numpy(par[t]))
                put(off[1], r.slopes); put(off[2], r.k_steps[t]); put(off[3], r.v_steps[t]); put(off[4], q)
            for redo in (False, True):
                for o in outs:
                    o.fill_(float("nan"))
                stack.step(t, has_slopes=True, redo=redo)
                torch.cuda.synchronize()
                for o, ref in zip(outs, refs):
                    assert torch.allclose(o.float(), ref.cpu().float(), atol=4e-3, rtol=2e-2)
        for h, r in zip(hs, ls):
            assert np.array_equal(h.get_ancestry(), r.h.get_ancestry())
            assert h.get_error() == 0
    finally:
        for r in ls:
            r.close()
        for h in hs:
            h.destroy()


def test_read_bandwidth_aid():
    buf = torch.zeros(1 << 30, dtype=torch.uint8, device="cuda")
    gbs = sk.read_bandwidth(buf, 5)
    assert 2000.0 < gbs < 9000.0, gbs                 # a B200 streams several TB/s; nothing reads faster than HBM3e
    with pytest.raises(sk.SegKVError):
        sk.read_bandwidth(buf[1:17], 1)               # not 16-byte aligned


def test_argument_and_state_errors():
    h = sk.SegKV(1, 2, 2, 2, 64, 16, 4, torch.float16)
    dev = "cuda"
    k = torch.zeros(2, 2, 64, dtype=torch.float16, device=dev)
    q = torch.zeros(2, 2, 64, dtype=torch.float16, device=dev)
    par = torch.zeros(2, dtype=torch.int32, device=dev)
    with pytest.raises(sk.SegKVError) as e:
        h.append(0, None, k, k)
    assert e.value.code == sk.SEGKV_ESTATE                      # no prefill yet
    with pytest.raises(sk.SegKVError) as e:
        h.prefill_write(torch.zeros(1, 17, 2, 64, dtype=torch.float16, device=dev),
                        torch.zeros(1, 17, 2, 64, dtype=torch.float16, device=dev))
    assert e.value.code == sk.SEGKV_ECAPACITY
    h.prefill_write(None, None)
    with pytest.raises(sk.SegKVError) as e:
        h.decode_sdpa(q)
    assert e.value.code == sk.SEGKV_ESTATE                      # nothing to attend to
    with pytest.raises(sk.SegKVError) as e:
        h.append(1, par, k, k)
    assert e.value.code == sk.SEGKV_ESTATE                      # wrong step
    for t in range(4):
        h.append(t, par if t else None, k, k)
    with pytest.raises(sk.SegKVError) as e:
        h.append(4, par, k, k)
    assert e.value.code == sk.SEGKV_ECAPACITY
    assert h.get_error() == 0
    for bad in (-2, 2):                                          # launch-shape knobs: values they do not know
        with pytest.raises(sk.SegKVError) as e:
            h.set_persistent(bad)
        assert e.value.code == sk.SEGKV_EINVAL
    with pytest.raises(sk.SegKVError) as e:
        h.set_tile(48)
    assert e.value.code == sk.SEGKV_EINVAL
    h.destroy()
    with pytest.raises(sk.SegKVError) as e:
        sk.SegKV(1, 2, 3, 2, 64, 16, 4, torch.float16)
    assert e.value.code == sk.SEGKV_EINVAL
    wide = sk.SegKV(1, 4, 8, 2, 64, 16, 4, torch.float16)       # 16 query columns per kv head
    with pytest.raises(sk.SegKVError) as e:
        wide.set_persistent(1)                                   # the persistent form takes at most 8
    assert e.value.code == sk.SEGKV_EINVAL
    with pytest.raises(sk.SegKVError) as e:
        wide.set_tile(32)                                        # and so does the small-CTA form
    assert e.value.code == sk.SEGKV_EINVAL
    wide.destroy()


def test_out_of_range_parent_is_clamped_and_flagged():
    w = wl.CONFIGS[0]
    par = wl.make_parents(w)
    bad = par.copy(); bad[3, 1] = 9; bad[4, 2] = -5
    clamped = par.copy(); clamped[3, 1] = w.beams - 1; clamped[4, 2] = 0
    r = Run(w, parents=bad)
    r.parents = clamped          # what the oracle should see
    try:
        r.advance_to(7)
        assert r.h.get_error() == sk.SEGKV_DEV_BAD_PARENT
        assert r.h.get_error() == 0                 # read clears
        assert np.array_equal(r.h.get_ancestry(), r.oracle_ancestry(7))
        out, q = r.decode()
        r.check(out, q, 7, all_pairs(w))
    finally:
        r.close()
