"""Pins for the CPU oracle: things the paper and the mathematics fix, computed
here WITHOUT the oracle's own code (numpy only), so that a dropped term, a
wrong sign or index, or a transposed operand in the oracle fails a test."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2401_05391_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- helpers
def bits(x: torch.Tensor) -> np.ndarray:
    return wl.to_bits(x)


def f64(x: torch.Tensor) -> np.ndarray:
    """Widen through torch, not through the oracle."""
    return x.detach().to(torch.float64).cpu().numpy()


def draw(shape, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(dtype)


def problem(B, W, H, Hkv, D, P, T, dtype=torch.float16, seed=0, parents=None):
    rng = np.random.default_rng(seed)
    q = draw((B * W, H, D), dtype, seed * 7 + 1)
    kp = draw((B, P, Hkv, D), dtype, seed * 7 + 2)
    vp = draw((B, P, Hkv, D), dtype, seed * 7 + 3)
    kr = draw((T, B * W, Hkv, D), dtype, seed * 7 + 4)
    vr = draw((T, B * W, Hkv, D), dtype, seed * 7 + 5)
    if parents is None:
        parents = rng.integers(0, W, size=(T, B * W)).astype(np.int32)
    return q, kp, vp, kr, vr, np.ascontiguousarray(parents, dtype=np.int32)


def run_oracle(q, kp, vp, kr, vr, parent, B, W, t, slopes=None, dtype="f16", **kw):
    H, D = q.shape[1], q.shape[2]
    Hkv = kp.shape[2]
    return oracle.decode_sdpa(dtype, B, W, H, Hkv, D, bits(q), bits(kp), bits(vp),
                              bits(kr) if kr is not None else None,
                              bits(vr) if vr is not None else None, parent, t,
                              slopes=slopes, **kw)


def softmax_rows(x):
    x = x - x.max(axis=-1, keepdims=True)
    e = np.exp(x)
    return e / e.sum(axis=-1, keepdims=True)


def copied_cache_attention(q_steps, kp, vp, kr, vr, parent, B, W, t, slopes=None):
    """The standard flow the paper replaces (Fig. 1): an explicit per-beam
    cache, re-ordered by index select with the beam indices at every step,
    then concatenated with the new key/value; dense attention on the copy."""
    H, D = q_steps.shape[1], q_steps.shape[2]
    Hkv = kp.shape[2]
    grp = H // Hkv
    Kp, Vp, Kr, Vr, Q = map(f64, (kp, vp, kr, vr, q_steps))
    # prefill: the prompt copied to every beam  [B*W, Hkv, P, D]
    kc = np.repeat(Kp.transpose(0, 2, 1, 3), W, axis=0)
    vc = np.repeat(Vp.transpose(0, 2, 1, 3), W, axis=0)
    for s in range(t + 1):
        if s > 0:
            glob = (np.arange(B * W) // W) * W + parent[s]      # global beam_idx
            kc, vc = kc[glob], vc[glob]
        kc = np.concatenate([kc, Kr[s][:, :, None, :]], axis=2)
        vc = np.concatenate([vc, Vr[s][:, :, None, :]], axis=2)
    L = kc.shape[2]
    out = np.empty((B * W, H, D))
    for h in range(H):
        k, v = kc[:, h // grp], vc[:, h // grp]                  # [B*W, L, D]
        sc = np.einsum("gd,gld->gl", Q[:, h], k) / np.sqrt(D)
        if slopes is not None:
            sc = sc + float(slopes[h]) * (np.arange(L) - (L - 1))[None, :]
        out[:, h] = np.einsum("gl,gld->gd", softmax_rows(sc), v)
    return out


# ------------------------------------------------- storage-format widening
def test_f16_widening_matches_numpy_for_every_bit_pattern():
    allbits = np.arange(65536, dtype=np.uint16)
    got = oracle.widen("f16", allbits)
    want = allbits.view(np.float16).astype(np.float64)
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])
    assert np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))


def test_bf16_widening_matches_torch_for_every_bit_pattern():
    allbits = np.arange(65536, dtype=np.uint16)
    got = oracle.widen("bf16", allbits)
    want = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok])


# ----------------------------------------------- P1: beams = 1 is causal MHA
@pytest.mark.parametrize("dtype,name", [(torch.float16, "f16"), (torch.bfloat16, "bf16")])
def test_single_beam_equals_last_row_of_causal_attention(dtype, name):
    B, W, H, Hkv, D, P, T = 2, 1, 3, 3, 16, 5, 4
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, dtype, seed=11)
    par[:] = 0
    t = T - 1
    got = run_oracle(q, kp, vp, kr, vr, par, B, W, t, dtype=name)
    L = P + T
    for b in range(B):
        for h in range(H):
            K = np.concatenate([f64(kp)[b, :, h], f64(kr)[:, b, h]], axis=0)      # [L, D]
            V = np.concatenate([f64(vp)[b, :, h], f64(vr)[:, b, h]], axis=0)
            # textbook causal self-attention over the whole sequence; earlier
            # positions get arbitrary queries, the last one gets q
            Q = np.random.default_rng(b * 10 + h).standard_normal((L, D))
            Q[-1] = f64(q)[b, h]
            S = Q @ K.T / np.sqrt(D)
            S[np.triu_indices(L, k=1)] = -np.inf
            O = softmax_rows(S) @ V
            np.testing.assert_allclose(got[b, h], O[-1], rtol=1e-12, atol=1e-13)


# ------------------------------------------- P2: copied-cache brute force
def test_equals_copied_cache_for_every_parent_table_w2():
    B, W, H, Hkv, D, P, T = 1, 2, 2, 2, 8, 3, 3
    q, kp, vp, kr, vr, _ = problem(B, W, H, Hkv, D, P, T, seed=3)
    # rows 1..T-1 matter: enumerate all W^(W*(T-1)) tables, row 0 arbitrary
    for combo in itertools.product(range(W), repeat=W * (T - 1)):
        par = np.zeros((T, B * W), dtype=np.int32)
        par[0] = 1  # must be ignored
        par[1:] = np.array(combo, dtype=np.int32).reshape(T - 1, W)
        for t in range(T):
            got = run_oracle(q, kp, vp, kr, vr, par, B, W, t)
            want = copied_cache_attention(q, kp, vp, kr, vr, par, B, W, t)
            np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("seed", range(6))
def test_equals_copied_cache_random(seed):
    rng = np.random.default_rng(100 + seed)
    B = int(rng.integers(1, 4)); W = int(rng.integers(1, 5))
    Hkv = int(rng.integers(1, 4)); grp = int(rng.integers(1, 3)); H = Hkv * grp
    D = int(rng.choice([4, 8, 16])); P = int(rng.integers(0, 9)); T = int(rng.integers(1, 9))
    dtype, name = ((torch.float16, "f16"), (torch.bfloat16, "bf16"))[seed % 2]
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, dtype, seed=seed)
    slopes = None
    if seed % 3 == 0:
        slopes = (2.0 ** (-8.0 * np.arange(1, H + 1) / H)).astype(np.float32)
    for t in range(T):
        got = run_oracle(q, kp, vp, kr, vr, par, B, W, t, slopes=slopes, dtype=name)
        want = copied_cache_attention(q, kp, vp, kr, vr, par, B, W, t, slopes=slopes)
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-12)


# ------------------------------------------------ P3: softmax rows sum to 1
def test_softmax_rows_sum_to_one_and_are_positive():
    B, W, H, Hkv, D, P, T = 2, 3, 4, 2, 16, 7, 5
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, seed=5)
    out, probs = run_oracle(q, kp, vp, kr, vr, par, B, W, T - 1, return_probs=True)
    assert probs.shape == (B * W, H, P + T)
    assert (probs > 0).all()
    np.testing.assert_allclose(probs.sum(-1), 1.0, rtol=0, atol=1e-14)


# -------------------------------------- P4: identical keys -> mean of values
def test_identical_keys_give_mean_of_selected_values():
    B, W, H, Hkv, D, P, T = 2, 4, 2, 2, 8, 6, 5
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, seed=9)
    key = draw((D,), torch.float16, 77)
    kp = key.expand_as(kp).contiguous()
    kr = key.expand_as(kr).contiguous()
    t = T - 1
    got = run_oracle(q, kp, vp, kr, vr, par, B, W, t)
    rows = oracle.ancestry(par, B, W, t)
    Vp, Vr = f64(vp), f64(vr)
    for g in range(B * W):
        for h in range(H):
            vals = np.concatenate([Vp[g // W, :, h], np.stack([Vr[s, rows[g, s], h] for s in range(T)])])
            np.testing.assert_allclose(got[g, h], vals.mean(0), rtol=1e-12, atol=1e-13)


# ------------------------------------------------ P5/P6/P7: the index table
def test_ancestry_closed_forms():
    B, W, T = 3, 4, 9
    t = T - 1
    j = np.tile(np.arange(W), B)
    base = np.repeat(np.arange(B) * W, W)
    ident = np.tile(j, (T, 1)).astype(np.int32)
    rows = oracle.ancestry(ident, B, W, t)
    assert np.array_equal(rows, np.tile((base + j)[:, None], (1, T)))
    zero = np.zeros((T, B * W), dtype=np.int32)
    rows = oracle.ancestry(zero, B, W, t)
    assert np.array_equal(rows[:, :t], np.tile(base[:, None], (1, t)))
    assert np.array_equal(rows[:, t], base + j)
    cyc = np.tile((j + 1) % W, (T, 1)).astype(np.int32)
    rows = oracle.ancestry(cyc, B, W, t)
    want = base[:, None] + (j[:, None] + (t - np.arange(T))[None, :]) % W
    assert np.array_equal(rows, want)


def test_ancestry_invariants_random():
    for seed in range(5):
        rng = np.random.default_rng(seed)
        B, W, T = int(rng.integers(1, 5)), int(rng.integers(1, 7)), int(rng.integers(1, 40))
        par = rng.integers(0, W, size=(T, B * W)).astype(np.int32)
        prev = None
        for t in range(T):
            rows = oracle.ancestry(par, B, W, t)
            g = np.arange(B * W)
            assert np.array_equal(rows[:, t], g)
            assert np.array_equal(rows // W, np.tile((g // W)[:, None], (1, t + 1)))   # stays in its request
            if prev is not None:                                                       # incremental form
                src = (g // W) * W + par[t]
                assert np.array_equal(rows[:, :t], prev[src])
            # sharing is prefix-closed: distinct rows per (request, step) never shrinks with s
            for b in range(B):
                cnt = [len(set(rows[b * W:(b + 1) * W, s].tolist())) for s in range(t + 1)]
                assert cnt == sorted(cnt)
            prev = rows


def test_ancestry_ignores_parent_row_zero():
    B, W, T = 2, 3, 6
    rng = np.random.default_rng(1)
    par = rng.integers(0, W, size=(T, B * W)).astype(np.int32)
    a = oracle.ancestry(par, B, W, T - 1)
    par2 = par.copy(); par2[0] = (par[0] + 1) % W
    assert np.array_equal(a, oracle.ancestry(par2, B, W, T - 1))


def test_tagged_rows_are_the_ones_selected():
    """Keys are zero so the softmax is uniform; each response value row carries
    its own (step, row) tag, so the output reveals exactly which rows were
    gathered: out*(P+T) = sum of tags along the ancestry."""
    B, W, H, D, P, T = 2, 4, 1, 2, 3, 7
    rng = np.random.default_rng(4)
    par = rng.integers(0, W, size=(T, B * W)).astype(np.int32)
    q = torch.zeros(B * W, H, D, dtype=torch.float16)
    kp = torch.zeros(B, P, H, D, dtype=torch.float16); vp = torch.zeros_like(kp)
    kr = torch.zeros(T, B * W, H, D, dtype=torch.float16)
    tag = torch.arange(T * B * W, dtype=torch.float32).reshape(T, B * W)          # < 2048: exact in fp16
    vr = torch.zeros_like(kr)
    vr[:, :, 0, 0] = tag.to(torch.float16)
    vr[:, :, 0, 1] = 1.0
    t = T - 1
    got = run_oracle(q, kp, vp, kr, vr, par, B, W, t)
    for g in range(B * W):
        cur, want = g % W, 0.0
        for s in range(t, -1, -1):                       # independent walk
            want += s * B * W + (g // W) * W + cur
            if s > 0:
                cur = int(par[s, (g // W) * W + cur])
        assert abs(got[g, 0, 0] * (P + T) - want) < 1e-9
        assert abs(got[g, 0, 1] * (P + T) - T) < 1e-12


# -------------------------------------------------- P8: Eq. 1-3, Fig. 4 text
def test_cache_size_formulas_reproduce_the_papers_gptj_numbers():
    vals = {}
    with open(os.path.join(GOLDEN, "kv_memory_gptj.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = int(v)
    tok = oracle.cache_token(vals["layers"], vals["heads"], vals["head_dim"], vals["elem_bytes"])
    assert tok == 524288.0
    std = oracle.cache_standard(vals["batch"], vals["beams"], vals["n_prompt"], vals["n_response"], tok)
    seg = oracle.cache_segment(vals["batch"], vals["beams"], vals["n_prompt"], vals["n_response"], tok)
    assert round(std / 1e9) == vals["standard_gb"]
    assert round(seg / 1e9) == vals["segment_gb"]
    # "about 63%" is the ratio of the two printed (rounded) figures, 86/137; unrounded it is 5/8
    assert round(100 * round(seg / 1e9) / round(std / 1e9)) == vals["segment_over_standard_percent"]
    assert seg / std == 0.625
    # the paper subtracts the rounded figures (137 - 86); unrounded gives 51.5
    assert vals["standard_gb"] - vals["segment_gb"] == vals["saved_gb"]
    assert abs((std - seg) / 1e9 - vals["saved_gb"]) < 1.0


def test_segment_cache_capacity_rounds_up_to_sixteen_steps():
    tok = oracle.cache_token(1, 2, 4, 2)
    a = oracle.cache_segment(3, 4, 10, 1, tok)
    b = oracle.cache_segment(3, 4, 10, 16, tok)
    c = oracle.cache_segment(3, 4, 10, 17, tok)
    assert a == b == 3 * (10 + 4 * 16) * tok
    assert c == 3 * (10 + 4 * 32) * tok


# ------------------------------------------------------------ P9: ALiBi
def test_alibi_zero_slopes_equal_none_and_constant_shift_is_invisible():
    B, W, H, Hkv, D, P, T = 1, 3, 4, 4, 8, 5, 4
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, seed=21)
    t = T - 1
    none = run_oracle(q, kp, vp, kr, vr, par, B, W, t)
    zero = run_oracle(q, kp, vp, kr, vr, par, B, W, t, slopes=np.zeros(H, np.float32))
    assert np.array_equal(none, zero)
    # bias slope*(kpos - qpos) differs from slope*kpos by a per-row constant:
    # compare with an independent computation that uses slope*kpos
    slopes = np.array([0.5, 0.25, 0.125, 0.0625], np.float32)
    got = run_oracle(q, kp, vp, kr, vr, par, B, W, t, slopes=slopes)
    rows = oracle.ancestry(par, B, W, t)
    for g in range(B * W):
        for h in range(H):
            K = np.concatenate([f64(kp)[0, :, h], np.stack([f64(kr)[s, rows[g, s], h] for s in range(T)])])
            V = np.concatenate([f64(vp)[0, :, h], np.stack([f64(vr)[s, rows[g, s], h] for s in range(T)])])
            sc = K @ f64(q)[g, h] / np.sqrt(D) + float(slopes[h]) * np.arange(P + T)
            np.testing.assert_allclose(got[g, h], softmax_rows(sc[None])[0] @ V, rtol=1e-11, atol=1e-12)


def test_alibi_huge_slope_selects_the_newest_row():
    B, W, H, Hkv, D, P, T = 1, 2, 2, 2, 8, 6, 3
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, seed=22)
    t = T - 1
    got = run_oracle(q, kp, vp, kr, vr, par, B, W, t, slopes=np.full(H, 1e4, np.float32))
    np.testing.assert_allclose(got, f64(vr)[t], rtol=0, atol=1e-12)


# -------------------------------------------------- P10: order, single key
def test_prompt_row_permutation_is_invisible_without_alibi():
    B, W, H, Hkv, D, P, T = 2, 2, 2, 1, 8, 9, 3
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, seed=31)
    perm = torch.from_numpy(np.random.default_rng(0).permutation(P))
    a = run_oracle(q, kp, vp, kr, vr, par, B, W, T - 1)
    b = run_oracle(q, kp[:, perm].contiguous(), vp[:, perm].contiguous(), kr, vr, par, B, W, T - 1)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_single_key_returns_its_value_and_prompt_only_decode():
    B, W, H, Hkv, D = 2, 3, 2, 2, 8
    q, kp, vp, _, _, _ = problem(B, W, H, Hkv, D, 1, 1, seed=41)
    got = run_oracle(q, kp, vp, None, None, None, B, W, -1)
    want = np.repeat(f64(vp)[:, 0], W, axis=0)             # [B*W, H, D]
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-15)
    # prompt-only decode over several keys = plain softmax attention
    q, kp, vp, _, _, _ = problem(B, W, H, Hkv, D, 5, 1, seed=42)
    got = run_oracle(q, kp, vp, None, None, None, B, W, -1)
    for g in range(B * W):
        for h in range(H):
            sc = f64(kp)[g // W, :, h] @ f64(q)[g, h] / np.sqrt(D)
            np.testing.assert_allclose(got[g, h], softmax_rows(sc[None])[0] @ f64(vp)[g // W, :, h],
                                       rtol=1e-12, atol=1e-13)


def test_no_prompt_response_only():
    B, W, H, Hkv, D, T = 1, 3, 1, 1, 4, 4
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, 0, T, seed=43)
    got = run_oracle(q, kp, vp, kr, vr, par, B, W, T - 1)
    want = copied_cache_attention(q, kp, vp, kr, vr, par, B, W, T - 1)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)


# ------------------------------- P11: identity parents = independent beams
def test_identity_parents_equal_independent_single_beam_problems():
    B, W, H, Hkv, D, P, T = 2, 3, 2, 2, 8, 4, 5
    q, kp, vp, kr, vr, _ = problem(B, W, H, Hkv, D, P, T, seed=51)
    ident = np.tile(np.tile(np.arange(W), B), (T, 1)).astype(np.int32)
    t = T - 1
    got = run_oracle(q, kp, vp, kr, vr, ident, B, W, t)
    # B*W requests with one beam each and the prompt duplicated per beam
    kp1 = kp.repeat_interleave(W, dim=0); vp1 = vp.repeat_interleave(W, dim=0)
    zero = np.zeros((T, B * W), dtype=np.int32)
    want = run_oracle(q, kp1, vp1, kr, vr, zero, B * W, 1, t)
    assert np.array_equal(got, want)


def test_gqa_head_mapping():
    """Query head h reads kv head h // (H/Hkv): expanding K/V to H heads gives
    the same result as the grouped call."""
    B, W, H, Hkv, D, P, T = 1, 2, 6, 2, 8, 4, 3
    q, kp, vp, kr, vr, par = problem(B, W, H, Hkv, D, P, T, seed=61)
    got = run_oracle(q, kp, vp, kr, vr, par, B, W, T - 1)
    rep = H // Hkv
    want = run_oracle(q, kp.repeat_interleave(rep, 2), vp.repeat_interleave(rep, 2),
                      kr.repeat_interleave(rep, 2), vr.repeat_interleave(rep, 2), par, B, W, T - 1)
    assert np.array_equal(got, want)


def test_oracle_rejects_global_parent_ids():
    B, W, T = 2, 2, 3
    par = np.array([[0, 1, 0, 1], [0, 1, 2, 3], [0, 0, 0, 0]], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.ancestry(par, B, W, T - 1)


# ------------------------------------------------------------------ prefill
def test_prefill_equals_textbook_causal_attention():
    B, N, H, Hkv, D = 2, 9, 4, 2, 16
    for dtype, name in ((torch.float16, "f16"), (torch.bfloat16, "bf16")):
        q = draw((B, N, H, D), dtype, 201); k = draw((B, N, Hkv, D), dtype, 202); v = draw((B, N, Hkv, D), dtype, 203)
        slopes = np.array([0.5, 0.25, 0.125, 0.0625], np.float32)
        for sl in (None, slopes):
            got = oracle.prefill_sdpa(name, B, H, Hkv, D, bits(q), bits(k), bits(v), slopes=sl)
            for b in range(B):
                for h in range(H):
                    S = f64(q)[b, :, h] @ f64(k)[b, :, h // (H // Hkv)].T / np.sqrt(D)
                    if sl is not None:
                        S = S + float(sl[h]) * (np.arange(N)[None, :] - np.arange(N)[:, None])
                    S[np.triu_indices(N, k=1)] = -np.inf
                    np.testing.assert_allclose(got[b, :, h], softmax_rows(S) @ f64(v)[b, :, h // (H // Hkv)],
                                               rtol=1e-12, atol=1e-13)


def test_prefill_row_is_the_decode_oracle_on_the_prefix():
    """Prefill position i = decode attention of one beam over the first i+1 prompt keys (the paper
    calls the prefill kernel the special case of the decode kernel), incl. the ALiBi convention."""
    B, N, H, Hkv, D = 2, 7, 2, 1, 8
    q = draw((B, N, H, D), torch.float16, 211); k = draw((B, N, Hkv, D), torch.float16, 212)
    v = draw((B, N, Hkv, D), torch.float16, 213)
    slopes = np.array([0.3, 0.7], np.float32)
    got = oracle.prefill_sdpa("f16", B, H, Hkv, D, bits(q), bits(k), bits(v), slopes=slopes)
    for i in (0, 3, N - 1):
        dec = oracle.decode_sdpa("f16", B, 1, H, Hkv, D, bits(q[:, i].contiguous()), bits(k[:, :i + 1].contiguous()),
                                 bits(v[:, :i + 1].contiguous()), None, None, None, -1, slopes=slopes)
        np.testing.assert_allclose(got[:, i], dec, rtol=1e-12, atol=1e-13)


def test_prefill_first_position_returns_its_own_value():
    B, N, H, Hkv, D = 1, 5, 2, 2, 8
    q = draw((B, N, H, D), torch.float16, 221); k = draw((B, N, Hkv, D), torch.float16, 222)
    v = draw((B, N, Hkv, D), torch.float16, 223)
    got = oracle.prefill_sdpa("f16", B, H, Hkv, D, bits(q), bits(k), bits(v), rows=[(0, 0, 0), (0, 0, 1)])
    np.testing.assert_allclose(got, f64(v)[0, 0], rtol=0, atol=1e-15)


# ------------------------------------------------------------ rotary embedding
def _complex_rotation(x, pos, base, style):
    """Independent statement of the rotary embedding: each pair is a complex number multiplied by
    exp(i * pos * base^(-2j/D)) (numpy complex arithmetic, not the oracle's formula)."""
    n, D = x.shape
    theta = base ** (-2.0 * np.arange(D // 2) / D)
    rot = np.exp(1j * pos[:, None] * theta[None, :])
    if style == "half":
        z = (x[:, :D // 2] + 1j * x[:, D // 2:]) * rot
        return np.concatenate([z.real, z.imag], axis=1)
    z = (x[:, 0::2] + 1j * x[:, 1::2]) * rot
    out = np.empty_like(x)
    out[:, 0::2], out[:, 1::2] = z.real, z.imag
    return out


@pytest.mark.parametrize("style", ["half", "interleaved"])
@pytest.mark.parametrize("dtype,tdt", [("f16", torch.float16), ("bf16", torch.bfloat16)])
def test_rope_equals_complex_multiplication_and_tables_are_the_closed_form(style, dtype, tdt):
    D, n, base = 64, 37, 10000.0
    x = draw((n, D), tdt, 500)
    pos = np.arange(n, dtype=np.float64) * 3 + 1
    cos_t, sin_t = wl.rope_tables(200, D, base)
    # the table generator against the closed form, entry by entry
    theta = base ** (-2.0 * np.arange(D // 2) / D)
    m = np.arange(200, dtype=np.float64)[:, None]
    assert np.allclose(cos_t.numpy(), np.cos(m * theta[None, :]), atol=6e-8, rtol=0)
    assert np.allclose(sin_t.numpy(), np.sin(m * theta[None, :]), atol=6e-8, rtol=0)
    idx = pos.astype(np.int64)
    got = oracle.widen(dtype, oracle.rope(dtype, bits(x), cos_t.numpy()[idx], sin_t.numpy()[idx], style)).reshape(n, D)
    want = _complex_rotation(f64(x), pos, base, style)
    ulp = 2.0 ** (-10 if dtype == "f16" else -7)
    assert np.all(np.abs(got - want) <= ulp * np.maximum(np.abs(want), 2.0 ** -14) + 1e-6)


@pytest.mark.parametrize("style", ["half", "interleaved"])
def test_rope_position_zero_is_identity_and_pairs_keep_their_norm(style):
    D, n = 32, 9
    x = draw((n, D), torch.float16, 501)
    one, zero = np.ones((n, D // 2)), np.zeros((n, D // 2))
    assert np.array_equal(oracle.rope("f16", bits(x), one, zero, style), bits(x))
    ang = np.random.default_rng(3).uniform(0, 6.28, (n, D // 2))
    y = oracle.widen("f16", oracle.rope("f16", bits(x), np.cos(ang), np.sin(ang), style)).reshape(n, D)
    xf = f64(x)
    if style == "half":
        nx, ny = xf[:, :D // 2] ** 2 + xf[:, D // 2:] ** 2, y[:, :D // 2] ** 2 + y[:, D // 2:] ** 2
    else:
        nx, ny = xf[:, 0::2] ** 2 + xf[:, 1::2] ** 2, y[:, 0::2] ** 2 + y[:, 1::2] ** 2
    assert np.allclose(nx, ny, rtol=4e-3, atol=1e-5)
    # a quarter turn maps (a, b) to (-b, a) exactly
    q = oracle.widen("f16", oracle.rope("f16", bits(x), zero, one, style)).reshape(n, D)
    if style == "half":
        assert np.array_equal(q[:, :D // 2], -xf[:, D // 2:]) and np.array_equal(q[:, D // 2:], xf[:, :D // 2])
    else:
        assert np.array_equal(q[:, 0::2], -xf[:, 1::2]) and np.array_equal(q[:, 1::2], xf[:, 0::2])


@pytest.mark.parametrize("style", ["half", "interleaved"])
def test_rope_scores_depend_on_the_position_difference_only(style):
    # <R_m q, R_n k> = <R_(m-n) q, k>: the property the embedding exists for (float64 inputs that are
    # exactly representable, so only the final rounding of the rotated rows differs)
    D, base = 16, 100.0
    q, k = draw((1, D), torch.float16, 502), draw((1, D), torch.float16, 503)
    cos_t, sin_t = [t.numpy().astype(np.float64) for t in wl.rope_tables(64, D, base)]

    def rot(x, m):
        return oracle.widen("f16", oracle.rope("f16", bits(x), cos_t[m:m + 1], sin_t[m:m + 1], style)).reshape(-1)
    for m, n in [(5, 2), (40, 37), (13, 10)]:
        a = float(rot(q, m) @ rot(k, n))
        b = float(rot(q, m - n) @ f64(k).reshape(-1))
        assert abs(a - b) <= 2e-2 * (np.abs(f64(q)).sum() * np.abs(f64(k)).max())


def test_narrow_rounds_to_nearest_even():
    # halfway cases and neighbours, against torch's conversions
    vals = np.array([1.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -2.5, 65504.0,
                     1e-5, 0.3333333333, -7.0625])
    t = torch.from_numpy(vals)
    assert np.array_equal(oracle.narrow("f16", vals), bits(t.to(torch.float16)))
    assert np.array_equal(oracle.narrow("bf16", vals), bits(t.to(torch.float32).to(torch.bfloat16)))
