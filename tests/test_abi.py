"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import os
import re

import pytest

import oracle
from paper_2401_05391_b200 import segkv as sk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"SEGKV_API[^;(]*?\b(segkv_\w+)\s*\(", text)
    return names


def test_header_declares_symbols():
    names = declared_symbols()
    assert len(names) >= 15 and len(set(names)) == len(names)


def test_every_declared_symbol_is_exported_and_bound():
    L = sk.lib()
    for name in declared_symbols():
        assert hasattr(L, name), f"{name} declared in include/ but not exported"
        assert name in sk.SIGNATURES, f"{name} has no Python binding signature"
    assert set(sk.SIGNATURES) == set(declared_symbols())


def test_storage_bytes_is_eq3_and_matches_the_papers_gptj_figure():
    # Eq. 3 per layer x 32 layers, GPT-J-6B of Table 1, BS=32, BW=4, 1024+1024, fp16 -> "86GB"
    per_layer = sk.segkv_storage_bytes(32, 4, 32, 128, 1024, 1024, sk.SEGKV_F16)
    assert round(32 * per_layer / 1e9) == 86
    tok = oracle.cache_token(32, 32, 128, 2)
    assert 32 * per_layer == oracle.cache_segment(32, 4, 1024, 1024, tok)
    assert sk.segkv_storage_bytes(0, 4, 32, 128, 1024, 1024, 0) == 0
    assert sk.segkv_storage_bytes(1, 4, 32, 128, 1024, 1024, 7) == 0


def test_error_strings():
    seen = {sk.segkv_strerror(c) for c in range(0, -7, -1)}
    assert len(seen) == 7
    assert "unknown" in sk.segkv_strerror(-99)


def test_null_handle_is_rejected_without_touching_a_gpu():
    L = sk.lib()
    assert L.segkv_steps(None) == sk.SEGKV_EINVAL
    assert L.segkv_reset(None, 1) == sk.SEGKV_EINVAL
    assert L.segkv_destroy(None) == sk.SEGKV_OK
    assert L.segkv_create(None, 1, 1, 1, 1, 64, 1, 1, 0) == sk.SEGKV_EINVAL
