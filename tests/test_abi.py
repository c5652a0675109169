"""Host-only checks of the C ABI: the library builds, loads and exports every declared symbol."""
import ctypes
import os
import re

import pytest

from paper_2412_04757_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ltri.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ltri_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    syms = declared_symbols()
    assert "ltri_create" in syms and "ltri_prefill_chunk" in syms and "ltri_decode_step" in syms
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in include/ltri.h but not exported"
    assert sorted(binding.EXPORTS) == syms


def test_struct_sizes_match_header(lib):
    # the C struct has 25 int32/float fields, one int64, seven pointers and two size_t with natural alignment
    assert ctypes.sizeof(binding.LtriParams) == 184
    assert ctypes.sizeof(binding.LtriStats) == 48


def test_arena_sizing_is_host_only_and_monotone(lib):
    p = binding.make_params(2, 8, 2, 4096, 256, 512, 64, 4)
    a = binding.ltri_arena_bytes(p)
    assert a > 2 * 2 * 2 * 4096 * 128 * 2            # at least the K/V cache
    p2 = binding.make_params(2, 8, 2, 8192, 256, 512, 64, 4)
    assert binding.ltri_arena_bytes(p2) > a


@pytest.mark.parametrize("kw", [
    dict(head_dim=64), dict(n_q_heads=6), dict(chunk=100), dict(chunk=2048), dict(top_k=0), dict(top_k=65),
    dict(n_sink=0), dict(n_sink=512), dict(window=0), dict(reps_per_span=9), dict(theta=1.5), dict(theta_mode=3),
    dict(max_tokens=0), dict(max_seqs=0), dict(n_kv_heads=3), dict(rep_mode=2), dict(rep_mode=1, max_reps=9),
    dict(rep_mode=1, min_reps=0), dict(rep_mode=1, min_reps=3, max_reps=2), dict(rep_mode=1, ratio_kind=3),
    dict(rep_mode=1, rep_lambda=-1.0), dict(unit_tokens=12), dict(unit_tokens=512), dict(nms_iou_milli=1000),
    dict(retrieval_head=[8]), dict(retrieval_head=[-2]), dict(retrieval_head=[1], retrieval_head_score=[-0.5]),
    dict(flags=4, unit_tokens=64), dict(flags=4, retrieval_head=[1]),
    dict(flags=8), dict(flags=8, unit_tokens=16, max_spans_per_region=4), dict(layer_theta=[1.5]),
    dict(flags=16, cache_units=8), dict(flags=16, unit_tokens=64, cache_units=3),
    dict(flags=16, unit_tokens=64, cache_units=129), dict(flags=16, unit_tokens=64, cache_units=8, score_decay=1.5),
    dict(flags=17, unit_tokens=64, cache_units=7), dict(layer_nms_iou_milli=[1000]), dict(layer_rep_lambda=[-1.0]),
])
def test_bad_parameters_are_rejected_on_the_host(lib, kw):
    base = dict(n_layers=1, n_q_heads=8, n_kv_heads=2, max_tokens=1024, chunk=256, window=512, n_sink=64, top_k=4)
    base.update(kw)
    p = binding.make_params(**base)
    assert binding.ltri_arena_bytes(p) == 0
    h = ctypes.c_void_p()
    p.arena = 256
    p.arena_bytes = 1 << 40
    assert lib.ltri_create(ctypes.byref(p), None, ctypes.byref(h)) == binding.LTRI_EINVAL


def test_create_rejects_null_small_or_misaligned_arena(lib):
    p = binding.make_params(1, 8, 2, 1024, 256, 512, 64, 4)
    h = ctypes.c_void_p()
    assert lib.ltri_create(ctypes.byref(p), None, ctypes.byref(h)) == binding.LTRI_EINVAL      # null arena
    p.arena, p.arena_bytes = 4096 + 8, 1 << 40
    assert lib.ltri_create(ctypes.byref(p), None, ctypes.byref(h)) == binding.LTRI_EINVAL      # misaligned
    p.arena, p.arena_bytes = 4096, 1024
    assert lib.ltri_create(ctypes.byref(p), None, ctypes.byref(h)) == binding.LTRI_ECAPACITY   # too small


def test_strerror(lib):
    assert binding.strerror(0) == "ok"
    for code in range(-6, 0):
        assert binding.strerror(code) != "unknown error"
    assert binding.strerror(-99) == "unknown error"


def test_product_package_does_not_reach_the_oracle():
    pkg = os.path.join(ROOT, "paper_2412_04757_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "inputs.py", f"{f} mentions the oracle"
