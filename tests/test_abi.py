"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header declares,
and its host-only entry points agree with the oracle."""
import os
import re

import numpy as np
import pytest

import paper_2609_17184_b200 as ls
from oracle import depths as dp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "loopspec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(loopspec_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(ls.lib, n), n
    assert sorted(ls.EXPORTS) == names


def test_pick_depths_matches_oracle():
    for a, b, R in [(1.03, 0.175, 32), (1.08, 0.207, 32), (1.0, 0.5, 16), (0.8, 0.3, 8), (1.03, 0.175, 4)]:
        d1s, d2s, d1, d2 = ls.pick_depths(a, b, R)
        o1, o2 = dp.optimal_depths(a, b, R)
        assert abs(d1s - o1) < 1e-6 * o1 and abs(d2s - o2) < 1e-6 * o2   # float arguments cross the ABI
        assert (d1, d2) == dp.snap_depths(float(__import__("numpy").float32(a)), float(__import__("numpy").float32(b)), R)
    with pytest.raises(ls.LoopSpecError):
        ls.pick_depths(-1.0, 0.2, 32)


def test_fit_envelope_matches_oracle_and_recovers_exact_power_laws():
    r = np.arange(1, 16, dtype=np.float64)
    a, b = ls.fit_envelope(0.2 * r ** -1.1)          # an exact power law is its own envelope
    assert abs(a - 1.1) < 1e-9 and abs(b - 0.2) < 1e-9
    rng = np.random.default_rng(4)
    for _ in range(40):
        n = int(rng.integers(3, 33))
        rr = np.arange(1, n + 1, dtype=np.float64)
        tv = rng.uniform(0.05, 0.4) * rr ** -rng.uniform(0.3, 2.0) * np.exp(rng.normal(0, 0.15, n))
        a, b = ls.fit_envelope(tv)
        ao, bo = dp.fit_envelope(tv)
        assert abs(a - ao) < 1e-9 * max(1, abs(ao)) and abs(b - bo) < 1e-9 * max(1, abs(bo))
        phi = b * rr ** -a
        assert (phi >= tv * (1 - 1e-12)).all() and a > 0       # an envelope: never below the measured profile
    with pytest.raises(ls.LoopSpecError):
        ls.fit_envelope([0.1, 0.2, 0.3])                       # never decreases: no positive exponent
    with pytest.raises(ls.LoopSpecError):
        ls.fit_envelope([0.1])
    with pytest.raises(ls.LoopSpecError):
        ls.fit_envelope([0.2, 0.0, 0.1])


def test_max_branches_matches_oracle_and_paper():
    assert ls.max_branches(32, 2, 8) == 249
    for R, d1, d2 in [(4, 1, 2), (4, 1, 3), (4, 1, 0), (4, 2, 0), (16, 2, 8), (32, 2, 10), (8, 2, 4)]:
        assert ls.max_branches(R, d1, d2) == dp.max_branches(R, d1, d2)
    assert ls.max_branches(4, 3, 0) == 0 and ls.max_branches(4, 1, 4) == 0 and ls.max_branches(8, 2, 5) == 0


def test_workspace_query_rejects_bad_shapes():
    import ctypes as C
    from paper_2609_17184_b200.binding import Model, Sched
    m = Model(512, 256, 4, 4, 64, 688, 0, 2, 0, 4, 0, 1, 1e-6, 1e4)
    s = Sched(1, 0, 0, 0, 1, 1, 0.0, 0, 1, 128, 0)
    assert ls.lib.loopspec_workspace_bytes(C.byref(m), C.byref(s)) > 0
    bad = Model(512, 250, 4, 4, 64, 688, 0, 2, 0, 4, 0, 1, 1e-6, 1e4)
    assert ls.lib.loopspec_workspace_bytes(C.byref(bad), C.byref(s)) == 0
    s2 = Sched(3, 0, 0, 0, 1, 1, 0.0, 0, 1, 128, 0)      # d1 does not divide R
    assert ls.lib.loopspec_workspace_bytes(C.byref(m), C.byref(s2)) == 0
    assert ls.linear_scratch_bytes(4, 256, 256) > 0 and ls.linear_scratch_bytes(4, 250, 256) == 0
