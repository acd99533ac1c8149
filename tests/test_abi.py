"""The C-ABI library loads without a GPU, exports every symbol the header declares, and its
host-only entry points validate arguments as the header says."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ms():
    from paper_2508_12801_b200 import binding
    return binding


def test_header_symbols_are_exported(ms):
    text = open(os.path.join(ROOT, "include", "maxscore.h")).read()
    declared = set(re.findall(r"\b(maxscore_[a-z_0-9]+)\s*\(", text))
    assert {"maxscore_route_fwd", "maxscore_route_bwd", "maxscore_dispatch", "maxscore_combine"} <= declared
    lib = C.CDLL(ms.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(ms.EXPORTS)


def test_struct_layouts_match_header(ms):
    assert C.sizeof(ms.Params) == 16 * 4 and ms.Params.softtopk_mode.offset == 13 * 4
    assert C.sizeof(ms.Stats) == 40 and ms.Stats.total_score.offset == 32
    assert C.sizeof(ms.DeviceBuffers) == 12 * 8


def test_capacity_formula(ms):
    # Sec. 2.3: C = cf * k * n / e, rounded up
    for (T, d, E, k, cf, want) in [(512, 256, 8, 2, 1.0, 128), (4096, 1024, 16, 2, 1.0, 512),
                                   (8192, 2048, 64, 8, 1.0, 1024), (16384, 2048, 64, 8, 1.25, 2560),
                                   (65536, 4096, 128, 8, 1.0, 4096), (7, 8, 4, 2, 1.0, 4)]:
        assert ms.capacity(ms.make_params(T, d, E, k, cf)) == want
    assert ms.capacity(ms.make_params(100, 8, 4, 2, 1.0, capacity=77)) == 77


def test_host_side_validation(ms):
    ok = ms.make_params(512, 256, 8, 2, io_dtype=ms.F32)
    assert ms.workspace_bytes(ok) > 0
    cases = [
        (ms.make_params(0, 256, 8, 2), 1),                       # non-positive size
        (ms.make_params(512, 256, 8, 2, t=0.0), 1),              # temperature must be > 0
        (ms.make_params(512, 256, 4, 5), 2),                     # k > E
        (ms.make_params(512, 256, 8, 2, capacity=100), 2),       # 8*100 < 1024
        (ms.make_params(512, 256, 256, 2), 6),                   # E above the supported limit
        (ms.make_params(512, 256, 16, 9), 6),                    # k above the supported limit
        (ms.make_params(512, 252, 8, 2, io_dtype=ms.BF16), 6),   # bf16 rows must be 16-byte multiples
        (ms.make_params(512, 256, 8, 2, score_mode=3), 1),
    ]
    for p, want in cases:
        with pytest.raises(ms.MaxScoreError) as ei:
            ms.workspace_bytes(p)
        assert ei.value.status == want
    n = C.c_size_t()
    lib = C.CDLL(ms.LIB_PATH)
    assert lib.maxscore_workspace_bytes(None, C.byref(n)) == 1
    assert lib.maxscore_workspace_bytes(C.byref(ok), None) == 1
    assert lib.maxscore_capacity(None) == -1
    # NULL context is rejected before any launch
    assert lib.maxscore_dispatch(None, None, None, None, None, None, None) == 1
    assert lib.maxscore_route_fwd(*([None] * 13)) == 1


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2508_12801_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f
