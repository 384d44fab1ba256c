"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates arguments, and counts retained/dropped tokens like the oracle."""

import ctypes
import itertools
import os
import re

import pytest

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "avggt.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(avggt_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    lib = binding.lib()
    for name in declared:
        assert getattr(lib, name) is not None
    assert re.fullmatch(r"\d+\.\d+\.\d+", P.avggt_version())


def test_params_struct_matches_header_layout():
    # 11 int32 + float + uint32, no padding
    assert ctypes.sizeof(P.AvggtParams) == 13 * 4


@pytest.mark.parametrize("sigma", (1, 2, 4, 6, 9))
@pytest.mark.parametrize("grid", [(37, 37), (16, 16), (28, 37), (3, 2), (1, 1), (5, 9)])
@pytest.mark.parametrize("kff", (False, True))
def test_kv_count_matches_oracle(sigma, grid, kff):
    p = P.make_params(7, grid[0], grid[1], 5, 16, 64, sigma, keep_first_frame=kff)
    cfg = orc.SGAConfig(7, grid[0], grid[1], 5, 16, 64, sigma, keep_first_frame=kff)
    assert P.avggt_kv_count(p) == orc.kv_count(cfg)


def test_benchmark_sizes():
    sizes = {(100, 4): (36600, 100800), (300, 6): (75600, 336600), (800, 9): (139200, 960000),
             (333, 1): (457542, 0), (333, 2): (235764, 221778)}
    for (n, s), want in sizes.items():
        assert P.avggt_kv_count(P.make_params(n, 37, 37, 5, 16, 64, s)) == want


def _code(**over):
    kw = dict(n_frames=4, grid_h=6, grid_w=6, n_special=5, n_heads=4, head_dim=64, sigma=4)
    kw.update(over)
    extra = {k: kw.pop(k) for k in ("tokens_per_frame",) if k in kw}
    p = P.make_params(**kw)
    for k, v in extra.items():
        setattr(p, k, v)
    m, nd = ctypes.c_int64(), ctypes.c_int64()
    return binding.lib().avggt_kv_count(ctypes.byref(p), ctypes.byref(m), ctypes.byref(nd))


def test_argument_validation_codes():
    assert _code() == 0
    assert _code(sigma=3) == -2 and _code(sigma=0) == -2 and _code(sigma=8) == -2      # not in the printed table
    assert _code(head_dim=128) == -2 and _code(batch=2) == -2 and _code(n_heads=33) == -2
    assert _code(n_frames=0) == -1 and _code(grid_h=0) == -1 and _code(n_special=-1) == -1
    assert _code(tokens_per_frame=40) == -1                                              # L != n_special + h*w
    assert _code(diag=2) == -1 and _code(mean_fill=3) == -1
    assert _code(softmax_scale=float("nan")) == -1
    p = P.make_params(4, 6, 6, 5, 4, 64, 4)
    p.flags = 6
    assert binding.lib().avggt_kv_count(ctypes.byref(p), None, None) == -1
    assert binding.lib().avggt_kv_count(None, None, None) == -1
    for code in range(-6, 1):
        assert binding.lib().avggt_strerror(code)
    assert b"unknown" in binding.lib().avggt_strerror(-99)


def test_frame_attention_work_item_limit_is_checked_on_the_host():
    """ceil(L / 256) * H * N work items must fit a 32-bit count: rejected before any device call."""
    p = P.make_params(1 << 26, 1, 1, 1, 32, 64, 4)     # 2 tokens per frame, 2^27 tokens, 2^31 work items
    lib = binding.lib()
    assert lib.avggt_kv_count(ctypes.byref(p), None, None) == 0
    assert lib.avggt_frame_attn(ctypes.byref(p), None, None, None, None, None, None, 0, None) == -2


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2512_02541_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", text, flags=re.M), f
                assert "avggt_oracle" not in text and "oracle/" not in text, f
    text = open(os.path.join(ROOT, "oracle", "avggt_oracle.py")).read()
    assert "import paper_2512_02541_b200" not in text and "from paper_2512_02541_b200" not in text
