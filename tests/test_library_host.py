"""Host-side checks that need no GPU: the shared library loads, exports every symbol the header
declares, and its planner agrees with the CPU checker to the last integer."""
import os
import re

import numpy as np
import pytest

from oracle import spindlekv_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, fn)).read(), flags=re.S)
            names |= set(re.findall(r"\b(spindlekv_[a-z_]+)\s*\(", text))
    return sorted(names)


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


def test_device_entry_points_reject_bad_arguments_before_touching_the_gpu():
    # argument checks come first in every entry point, so they can be exercised without a device
    import ctypes as C
    from paper_2507_06517_b200 import binding as B
    lib = B._lib
    cfg = B.Config(4, 8, 2, 128, 32, 2, budget_tokens=300.0).c()
    good = B._Tensor(256, B.BF16, 8, 8, 8, 8)          # an aligned, non-null address that is never dereferenced
    odd = B._Tensor(264, B.BF16, 8, 8, 8, 8)           # not 16-byte aligned
    f32 = B._Tensor(256, B.F32, 8, 8, 8, 8)
    batch = B._Batch(1, 1, 1024, 1024, None, None, 0)
    both = B._Batch(1, 1, 1024, 1024, 256, 256, 0)     # packed and per-layer lengths at once
    p = C.c_void_p(256)
    assert lib.spindlekv_evict_deep(C.byref(cfg), C.byref(batch), good, good, None, p, p, p, p, 1 << 20, None) == B.INVALID_ARG
    assert lib.spindlekv_evict_deep(C.byref(cfg), C.byref(batch), odd, good, p, p, p, p, p, 1 << 20, None) == B.INVALID_ARG
    assert lib.spindlekv_evict_deep(C.byref(cfg), C.byref(batch), good, f32, p, p, p, p, p, 1 << 20, None) == B.UNSUPPORTED
    assert lib.spindlekv_evict_deep(C.byref(cfg), C.byref(both), good, good, p, p, p, p, p, 1 << 20, None) == B.INVALID_ARG
    assert lib.spindlekv_codebook_shallow(C.byref(cfg), C.byref(both), good, 0.98, p, p, p, p, None, p, 1 << 20, None) == B.INVALID_ARG
    assert lib.spindlekv_codebook_shallow(C.byref(cfg), C.byref(batch), good, 0.98, None, p, p, p, None, p, 1 << 20, None) == B.INVALID_ARG
    assert lib.spindlekv_codebook_shallow(C.byref(cfg), C.byref(batch), good, 0.98, p, p, p, p, C.c_void_p(260), p, 1 << 20, None) == B.INVALID_ARG  # adjacency not 16-byte aligned
    bad_dim = B.Config(4, 8, 2, 96, 32, 2, budget_tokens=300.0).c()
    assert lib.spindlekv_codebook_shallow(C.byref(bad_dim), C.byref(batch), good, 0.98, p, p, p, p, None, p, 1 << 20, None) == B.UNSUPPORTED
    assert lib.spindlekv_compact(C.byref(batch), 2, 128, good, None, p, None, good, None, None) == B.INVALID_ARG
    assert lib.spindlekv_compact(C.byref(batch), 2, 128, good, p, p, None, f32, None, None) == B.UNSUPPORTED
    assert lib.spindlekv_reconstruct(C.byref(batch), 2, 128, good, None, p, good, None) == B.INVALID_ARG
    assert lib.spindlekv_reconstruct(C.byref(batch), 2, 96, good, p, p, good, None) == B.UNSUPPORTED
    assert lib.spindlekv_union_lists(1, 2, 2, 4, 0, 100, 60, p, p, 400, 200, p, p, None) == B.INVALID_ARG   # 2 x 60 > 100
    assert lib.spindlekv_union_lists(1, 1, 2, 4, 1, 100, 100, None, p, 400, 400, p, p, None) == B.INVALID_ARG
    assert lib.spindlekv_match_workspace_bytes(C.byref(both), 2) == 0
    assert lib.spindlekv_match_workspace_bytes(C.byref(batch), 2) >= 8 * 2 * 1024
    assert lib.spindlekv_codebook_match(C.byref(batch), 2, 128, good, good, p, 0, 0.98, p, p, p, p, p, 1 << 20, None) == B.INVALID_ARG
    assert lib.spindlekv_codebook_match(C.byref(batch), 2, 128, good, f32, p, 64, 0.98, p, p, p, p, p, 1 << 20, None) == B.UNSUPPORTED
    assert lib.spindlekv_codebook_append(C.byref(batch), 2, 128, good, p, p, p, p, p, None, good, 64, p, p, None) == B.INVALID_ARG
    assert lib.spindlekv_evict_deep_noalloc(C.byref(cfg), C.byref(batch), good, good, None, p, p, p, None) == B.INVALID_ARG
    assert lib.spindlekv_poll_status(None, p, None) == B.INVALID_ARG


def test_allocation_free_entry_point_checks_its_arguments_like_the_ordinary_one():
    # every rejection below comes back before anything is enqueued (no device is needed to see it): a
    # misaligned base or an odd stride would otherwise reach the 16-byte loads of the kernels
    import ctypes as C
    from paper_2507_06517_b200 import binding as B
    lib = B._lib
    cfg = B.Config(4, 8, 2, 128, 32, 2, budget_tokens=300.0).c()
    batch = B._Batch(1, 1, 1024, 1024, None, None, 0)
    p = C.c_void_p(256)
    good = B._Tensor(256, B.BF16, 8, 8, 8, 8)

    def call(K=good, Q=good, b=batch, c=cfg):
        return lib.spindlekv_evict_deep_noalloc(C.byref(c), C.byref(b), K, Q, p, p, p, p, None)

    assert call(K=B._Tensor(264, B.BF16, 8, 8, 8, 8)) == B.INVALID_ARG          # base not 16-byte aligned
    assert call(Q=B._Tensor(256, B.BF16, 8, 8, 8, 12)) == B.INVALID_ARG         # token stride not a multiple of 8
    assert call(K=B._Tensor(256, 7, 8, 8, 8, 8)) == B.INVALID_ARG               # unknown dtype
    assert call(Q=B._Tensor(256, B.F32, 8, 8, 8, 8)) == B.UNSUPPORTED           # K and Q of different types
    assert call(b=B._Batch(1, 2, 1024, 1024, None, None, 0)) == B.INVALID_ARG   # total_len != n_seqs * max_len
    assert call(b=B._Batch(1, 1, 1024, 1024, 256, 256, 0)) == B.INVALID_ARG     # packed and per-layer lengths at once
    assert call(b=B._Batch(0, 1, 1024, 1024, None, None, 0)) == B.INVALID_ARG   # no layers
    assert call(c=B.Config(4, 8, 2, 96, 32, 2, budget_tokens=300.0).c()) == B.UNSUPPORTED
    # fp32 inputs run on the CUDA-core kernels, whose row statistics must fit the fixed scratch
    f32 = B._Tensor(256, B.F32, 8, 8, 8, 8)
    big = B._Batch(16, 1, 16384, 16384, None, None, 0)
    assert B.spindlekv_workspace_bytes(B.Config(4, 8, 2, 128, 32, 2, budget_tokens=300.0),
                                       B.Batch(16, 1, 16384, 16384), B.WS_EVICT) > B.NOALLOC_SCRATCH_BYTES
    assert call(K=f32, Q=f32, b=big) == B.WORKSPACE_TOO_SMALL


def test_limits_can_be_tightened_and_restored():
    from paper_2507_06517_b200 import binding as B
    defaults = [B.spindlekv_get_tuning(k) for k in range(4)]
    assert defaults[B.TUNE_RECORDS_PER_TILE] == 512 and defaults[B.TUNE_SIM_BLOCK_PAIRS] == 0
    try:
        B.spindlekv_set_tuning(B.TUNE_RECORDS_PER_TILE, 7)
        B.spindlekv_set_tuning(B.TUNE_GREEDY_ROUND_CAP, 1)
        assert B.spindlekv_get_tuning(B.TUNE_RECORDS_PER_TILE) == 7 and B.spindlekv_get_tuning(B.TUNE_GREEDY_ROUND_CAP) == 1
        B.spindlekv_set_tuning(B.TUNE_SIM_BLOCK_PAIRS, 3)
        assert B.spindlekv_get_tuning(B.TUNE_SIM_BLOCK_PAIRS) == 3
        B.spindlekv_set_tuning(B.TUNE_RECORDS_PER_TILE, 100000)      # never above what the workspace is sized for
        assert B.spindlekv_get_tuning(B.TUNE_RECORDS_PER_TILE) == 512
        with pytest.raises(B.SpindleKVError):
            B.spindlekv_set_tuning(99, 1)
        assert B.spindlekv_get_tuning(99) == -1
    finally:
        for k in range(4):
            B.spindlekv_set_tuning(k, -1)
    assert [B.spindlekv_get_tuning(k) for k in range(4)] == defaults
    # the self-tests check their arguments before launching anything
    assert B._lib.spindlekv_selftest_mbarrier_timeout(None, 100, None) == B.INVALID_ARG
    assert B._lib.spindlekv_selftest_mbarrier_timeout(256, 0, None) == B.INVALID_ARG


def test_reserve_ratio_matches_checker():
    from paper_2507_06517_b200 import binding as B
    rng = np.random.default_rng(5)
    for _ in range(100):
        h = int(rng.integers(1, 33))
        l = int(rng.integers(64, 40000))
        kept = int(rng.integers(1, l + 1))
        ek, ev = rng.integers(1, kept + 1, size=h), rng.integers(1, kept + 1, size=h)
        assert B.spindlekv_reserve_ratio(l, kept, ek, ev) == O.reserve_ratio_layer(l, kept, ek, ev)
    with pytest.raises(B.SpindleKVError):
        B.spindlekv_reserve_ratio(100, 0, [1], [1])


def test_decode_entry_points_check_their_arguments():
    import ctypes as C
    from paper_2507_06517_b200 import binding as B
    lib = B._lib
    batch = B._Batch(1, 1, 1024, 1024, None, None, 0)
    packed = B._Batch(1, 1, 1024, 1024, 256, None, 0)
    good, f32 = B._Tensor(256, B.BF16, 8, 8, 8, 8), B._Tensor(256, B.F32, 8, 8, 8, 8)
    p = C.c_void_p(256)

    def call(b=batch, hq=8, hkv=2, d=128, q=good, ck=good, cv=good, table=p, npos=64, ws=p):
        return lib.spindlekv_decode_attend(C.byref(b), hq, hkv, d, q, p, ck, p, p, cv, p, p, None, table, npos, p, ws, 1 << 20, None)

    assert call(b=packed) == B.INVALID_ARG            # equal-length form only
    assert call(hq=7) == B.INVALID_ARG                # query heads must divide over the KV heads
    assert call(table=None) == B.INVALID_ARG
    assert call(ws=C.c_void_p(260)) == B.INVALID_ARG
    assert call(ck=f32) == B.UNSUPPORTED              # one dtype for q and both CodeBooks
    assert call(d=96) == B.UNSUPPORTED
    assert call(hq=32, hkv=2) == B.UNSUPPORTED        # more than 8 query heads per KV head
    assert B.spindlekv_rope_table_bytes(128, 4096) == 4096 * 64 * 8
    assert B.spindlekv_rope_table_bytes(100, 4096) == 0
    assert lib.spindlekv_rope_table(128, 0, 10000.0, p, None) == B.INVALID_ARG
    assert lib.spindlekv_decode_workspace_bytes(C.byref(packed), 8, 2, 128) == 0
    assert lib.spindlekv_decode_workspace_bytes(C.byref(batch), 8, 2, 128) >= 4 * 130 * 4 * 2
