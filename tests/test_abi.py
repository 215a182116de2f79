"""Host-side checks of the C-ABI library: it builds, loads, exports every declared symbol, validates arguments
and answers the size queries like the oracle's counting rule.  No GPU needed (no compute call is made)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import sla_oracle as orc
from paper_2605_11354_b200 import binding as lt
from paper_2605_11354_b200 import build as lb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    lb.build()
    return lt.lib()


def declared_symbols():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"LITE3R_API[^;(]*?\b(lite3r_\w+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported(built_library):
    names = declared_symbols()
    assert len(names) >= 9 and set(lt.EXPORTS) <= set(names)
    for name in names:
        assert hasattr(built_library, name), name


def test_class_counts_match_the_counting_rule():
    g = np.random.default_rng(0)
    cases = [(8, 0.25, 0.5), (172, 0.10, 0.60), (687, 0.05, 0.75), (172, 0.08, 0.70), (2147, 0.02, 0.6),
             (2147, 1.0, 0.0), (10, 0.0, 1.0), (2, 0.25, 0.0), (10, 0.6, 0.9)]
    cases += [(int(g.integers(1, 3000)), float(g.random()), float(g.random())) for _ in range(300)]
    for nb, crit, neg in cases:
        shape = lt.Shape(1, 1, nb * 64 - 5 if nb * 64 > 5 else 1, 64, 64)
        cls_b, crit_b, marg_b, kc, km, kn = lt.lite3r_plan_sizes(shape, crit, neg)
        assert (kc, km, kn) == orc.class_counts(nb, crit, neg), (nb, crit, neg)
        assert cls_b == nb * nb and crit_b == nb * kc * 4 and marg_b == nb * km * 4


def test_size_queries():
    shape = lt.Shape(4, 16, 21984, 64, 128)
    codes, scales, colsum = lt.lite3r_fp8_sizes(shape)
    assert codes == 4 * 16 * 172 * 128 * 64 and scales == 4 * 16 * 172 * 4 and colsum == 4 * 16 * 172 * 64 * 4
    plain = lt.lite3r_forward_workspace(shape, 0.08, 0.7)
    planned = lt.lite3r_forward_workspace_planned(shape, 0.08, 0.7)
    tiles = 4 * 16 * 172
    # with the plan inside, the class bytes and the critical lists (14 of 172 blocks) come on top
    assert plain > 0 and planned >= plain + tiles * 172 + tiles * 14 * 4
    off = lt.lite3r_workspace_layout(shape, 0.08, 0.7, plan_inside=True)
    assert off[0] == 0 and list(off) == sorted(off) and off[4] == plain and off[5] >= off[4] + tiles * 172
    assert off[1] - off[0] >= tiles * 4160 * 2 and off[2] - off[1] >= tiles * 64 * 64 * 2
    assert off[3] - off[2] >= tiles * 64 * 4 and off[4] - off[3] >= tiles * 128 * 64 * 2
    assert lt.lite3r_workspace_layout(shape, 0.08, 0.7)[:4] == off[:4]


def test_static_scratch_tile_limits():
    """The 32 MiB array holds 1344 tiles at block 64 and 1012 at block 128 (what the header says)."""
    for block, fits in ((64, 1344), (128, 1012)):
        assert lt.lite3r_forward_workspace(lt.Shape(1, 1, fits * block, 64, block), 0.1, 0.6) <= lt.STATIC_SCRATCH_BYTES
        assert lt.lite3r_forward_workspace(lt.Shape(1, 1, (fits + 1) * block, 64, block), 0.1, 0.6) > lt.STATIC_SCRATCH_BYTES


@pytest.mark.parametrize("shape,status", [
    ((1, 1, 100, 32, 64), "unsupported"), ((1, 1, 100, 64, 32), "unsupported"), ((0, 1, 100, 64, 64), "invalid"),
    ((1, 1, 0, 64, 64), "invalid")])
def test_bad_shapes_are_rejected(shape, status):
    with pytest.raises(lt.Lite3rError, match=status):
        lt.lite3r_fp8_sizes(lt.Shape(*shape))


def test_bad_fractions_and_null_pointers_are_rejected(built_library):
    shape = lt.Shape(1, 1, 100, 64, 64)
    for crit, neg in ((-0.1, 0.5), (1.5, 0.0), (0.5, float("nan"))):
        with pytest.raises(lt.Lite3rError, match="invalid"):
            lt.lite3r_plan_sizes(shape, crit, neg)
    # compute calls with null buffers fail on validation before anything is enqueued
    t = lt.Tensor(None, 0, 6400, 6400, 64)
    assert built_library.lite3r_quantize_fp8(C.byref(t), C.byref(shape), lt.Fp8(None, None, None), None) == 1
    f = lt.Fp8(None, None, None)
    p = lt.Plan(None, None, None, 0, 0, 0)
    assert built_library.lite3r_sla_plan(C.byref(f), C.byref(f), C.byref(shape), 0.5, 0.2, C.byref(p), None) == 1
    assert built_library.lite3r_sla_forward(C.byref(f), C.byref(f), C.byref(f), None, 0, C.byref(shape), 0.5, 0.2, 0,
                                            C.byref(p), None, 0, 0, 0, 64, None, 0, None, None) == 1
    # no plan: the fractions are validated instead, and q / k must then carry column sums
    assert built_library.lite3r_sla_forward(C.byref(f), C.byref(f), C.byref(f), None, 0, C.byref(shape), 1.5, 0.2, 0,
                                            None, None, 0, 0, 0, 64, None, 0, None, None) == 1
    assert built_library.lite3r_status_string(3) == b"workspace too small"
