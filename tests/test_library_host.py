"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header
declares, and its planner agrees with the CPU checker to the last integer."""
import os
import re

import numpy as np
import pytest

from oracle import spindlekv_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "spindlekv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spindlekv_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2507_06517_b200 import binding as B
    names = _declared()
    assert {"spindlekv_plan_layers", "spindlekv_evict_deep", "spindlekv_codebook_shallow",
            "spindlekv_compact"} <= set(names)
    for n in names:
        assert hasattr(B._lib, n), n
        assert hasattr(B, n) or n == "spindlekv_status_string", f"binding lacks {n}"


def test_planner_matches_checker():
    from paper_2507_06517_b200 import binding as B
    rng = np.random.default_rng(3)
    for _ in range(200):
        m = int(rng.integers(1, 48))
        ns = int(rng.integers(-1, m + 1))   # -1: every layer evicts, then builds CodeBooks
        Bn = int(rng.integers(1, 5))
        w = int(rng.choice([16, 32, 64]))
        lens = [int(x) for x in rng.integers(w + 200, 40000, size=Bn)]
        if rng.random() < 0.5:
            kw = dict(budget_tokens=float(rng.integers(int(0.06 * (min(lens) - w)) + w + 2, min(lens))))
            okw = dict(budget_tokens=kw["budget_tokens"])
        else:
            r = float(rng.uniform(0.08, 1.0))
            kw = dict(reserve_ratio=r)
            okw = dict(reserve_ratio=r)
        cfg = B.Config(m, 8, 2, 128, w, ns, **kw)
        try:
            want = O.plan_layers(m, ns, lens, w, 0.05, **okw)
        except O.BudgetError:
            with pytest.raises(B.SpindleKVError) as e:
                B.spindlekv_plan_layers(cfg, lens)
            assert e.value.status == B.BUDGET
            continue
        mode, ratio, k = B.spindlekv_plan_layers(cfg, lens)
        assert np.array_equal(mode, want[0])
        assert np.array_equal(ratio, want[1])  # same IEEE operations in the same order
        assert np.array_equal(k, want[2])


def test_planner_rejects_bad_arguments():
    from paper_2507_06517_b200 import binding as B
    cfg = B.Config(4, 8, 2, 128, 32, 2, budget_tokens=64.0)
    with pytest.raises(B.SpindleKVError) as e:
        B.spindlekv_plan_layers(cfg, [32])  # not longer than the window
    assert e.value.status == B.INVALID_ARG
    with pytest.raises(B.SpindleKVError) as e:
        B.spindlekv_plan_layers(B.Config(4, 8, 3, 128, 32, 2, budget_tokens=64.0), [512])  # 8 % 3 != 0
    assert e.value.status == B.INVALID_ARG
    with pytest.raises(B.SpindleKVError) as e:
        B.spindlekv_plan_layers(B.Config(4, 8, 2, 128, 32, 2, budget_tokens=40.0), [4096])  # r_c <= beta
    assert e.value.status == B.BUDGET


def test_workspace_bytes_is_zero_on_bad_input_and_monotone():
    from paper_2507_06517_b200 import binding as B
    cfg = B.Config(4, 8, 2, 128, 32, 2, budget_tokens=300.0)
    assert B.spindlekv_workspace_bytes(cfg, B.Batch(1, 1, 16, 16), B.WS_EVICT) == 0  # shorter than the window
    a = B.spindlekv_workspace_bytes(cfg, B.Batch(1, 1, 1024, 1024), B.WS_CODEBOOK)
    b = B.spindlekv_workspace_bytes(cfg, B.Batch(2, 1, 1024, 1024), B.WS_CODEBOOK)
    c = B.spindlekv_workspace_bytes(cfg, B.Batch(1, 1, 2048, 2048), B.WS_CODEBOOK)
    assert 0 < a < b and a < c
    # the adjacency bit matrix dominates: N^2/8 bytes per unit
    assert a >= 2 * 1024 * 1024 // 8
