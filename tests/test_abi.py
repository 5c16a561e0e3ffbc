"""CPU-side checks of the CUDA library: it builds, loads without a GPU, exports every symbol the
public header declares, and its host planner cuts tensors into tiles that cover every element
exactly once.  No kernel is launched here."""
import os
import re

import numpy as np
import pytest

import paper_2501_07161_b200 as q
from paper_2501_07161_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TILE = 16384


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "qv2.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(qv2_[a-z_0-9]+)\s*\(", hdr))
    assert {"qv2_calibrate", "qv2_quant_metrics", "qv2_rank_layers"} <= declared
    L = q.lib()
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} is declared in qv2.h but not exported by libqv2.so"
    assert declared == set(B.EXPORTS)


def test_struct_layouts_match_the_header():
    import ctypes as C
    assert C.sizeof(B.TensorDesc) == 64 and B.TensorDesc.percentile.offset == 56
    assert C.sizeof(B.RankCfg) == 48
    assert C.sizeof(B.SweepBuffers) == 16 * 8 and C.sizeof(B.HostResults) == 6 * 8


def test_status_strings():
    L = q.lib()
    assert L.qv2_status_string(0) == b"QV2_OK"
    for s in range(-8, 0):
        assert L.qv2_status_string(s).startswith(b"QV2_ERR_")


def _desc(outer, ch, inner, per_channel, ptr=4096, percentile=None):
    d = q.make_desc(None, None, outer, ch, inner, q.PER_CHANNEL if per_channel else q.PER_TENSOR,
                    q.ASYM_U8, q.PERCENTILE if percentile is not None else q.MINMAX, percentile or 0.0)
    d.x = ptr
    return d


@pytest.mark.parametrize("outer,ch,inner,pc", [(1, 1, 1, False), (1, 1, 5 * TILE + 3, False),
                                               (1, 960, 9, True), (1, 64, 576, True), (64, 256, 3136, True), (2, 9, 127, True), (2, 9, 128, True), (1, 7, 4096, True), (5, 3, 9000, True), (1, 4, TILE - 1, True),
                                               (1, 3, 25088, True), (3, 5, 4095, True), (2, 3, 40000, True),
                                               (1, 1, TILE, True), (4, 1, 1, True)])
def test_tiles_cover_every_element_once(outer, ch, inner, pc):
    descs = q.desc_array([_desc(outer, ch, inner, pc), _desc(1, 1, 100, False)])
    tiles = B.plan_tiles(descs)
    n = outer * ch * inner
    mine = [t for t in tiles if t[0] == 0]
    pos = 0
    for tensor, begin, count, kind in mine:
        assert begin == pos and 0 < count <= TILE
        if kind == 1:                       # whole rows only, as many as fit a tile
            assert begin % inner == 0 and count % inner == 0 and inner < TILE
            assert count // inner == max(1, TILE // inner) or begin + count == n
        elif pc:                            # one-group tile never crosses a row
            assert begin // inner == (begin + count - 1) // inner
        pos += count
    assert pos == n
    assert [t for t in tiles if t[0] == 1] == [(1, 0, 100, 0)]


def test_group_count_and_plan_errors():
    L = q.lib()
    descs = q.desc_array([_desc(1, 64, 576, True), _desc(8, 3, 10, False), _desc(2, 5, 7, True)])
    assert L.qv2_group_count(descs, 3) == 64 + 1 + 5
    bad = _desc(1, 1, 10, False); bad.scheme = 9
    assert L.qv2_debug_plan_tiles(q.desc_array([bad]), 1, None, 0) == -1
    bad = _desc(1, 1, 10, False); bad.x = 4098
    assert L.qv2_debug_plan_tiles(q.desc_array([bad]), 1, None, 0) == -3
    bad = _desc(1, 1, 10, False); bad.x = None
    assert L.qv2_debug_plan_tiles(q.desc_array([bad]), 1, None, 0) == -2
    bad = _desc(1 << 40, 1 << 30, 1 << 20, False)
    assert L.qv2_debug_plan_tiles(q.desc_array([bad]), 1, None, 0) == -4
    bad = _desc(1, 1, 10, False, percentile=2.0)
    assert L.qv2_debug_plan_tiles(q.desc_array([bad]), 1, None, 0) == -1
    assert L.qv2_debug_plan_tiles(q.desc_array([_desc(1, 1, 10, False)]), 0, None, 0) == -4
    empty = _desc(0, 4, 10, True); empty.x = None
    assert L.qv2_debug_plan_tiles(q.desc_array([empty]), 1, None, 0) == 0
    # per-group percentile: same argument checks, histograms only for per-channel tensors that ask
    g = _desc(2, 5, 100, True, percentile=0.99); g.range = q.PERCENTILE_GROUP
    t = _desc(2, 5, 100, False, percentile=0.99); t.range = q.PERCENTILE_GROUP
    p = _desc(2, 7, 100, True, percentile=0.99)
    assert L.qv2_group_hist_count(q.desc_array([g, t, p, g]), 4) == 10
    assert L.qv2_debug_plan_tiles(q.desc_array([g, t, p]), 3, None, 0) > 0
    bad = _desc(2, 5, 100, True, percentile=-0.1); bad.range = q.PERCENTILE_GROUP
    assert L.qv2_debug_plan_tiles(q.desc_array([bad]), 1, None, 0) == -1
    bad = _desc(1, 1, 10, False); bad.range = 4
    assert L.qv2_debug_plan_tiles(q.desc_array([bad]), 1, None, 0) == -1
    huge = _desc(1 << 24, 1 << 12, 100, True, percentile=0.9); huge.range = q.PERCENTILE_GROUP
    assert L.qv2_debug_plan_tiles(q.desc_array([huge]), 1, None, 0) == -4      # refused before any table is built
    assert L.qv2_debug_plan_tiles(q.desc_array([_desc(1, 1, 1 << 50, False)]), 1, None, 0) == -4
    assert L.qv2_debug_plan_tiles(q.desc_array([_desc(1 << 30, 4, 5000, True)]), 1, None, 0) == -4


def test_no_gpu_means_a_loud_failure_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    import ctypes as C
    h = C.c_void_p()
    assert q.lib().qv2_create(C.byref(h), 0, None) == -6      # QV2_ERR_CUDA
    with pytest.raises(Exception):
        q.Context(0)
