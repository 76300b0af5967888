"""Host-side checks that need no GPU: the library loads and exports every symbol the
header declares, argument validation, and the selector DP against the oracle's brute force."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2312_14227_b200 as et
import workloads as wl
from oracle import elastic_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    with open(os.path.join(ROOT, "include", "et.h")) as f:
        header = f.read()
    declared = set(re.findall(r"\b(et_[a-z_0-9]+)\s*\(", header))
    assert len(declared) >= 18
    lib = ctypes.CDLL(et.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in et.h but not exported"
    assert declared == set(et.EXPORTED_SYMBOLS)


def test_status_strings():
    assert et.et_status_string(0) == "ok"
    assert "timed out" in et.et_status_string(et.ET_ERR_TIMEOUT)


def _err(layers, M=16, dtype=et.ET_F32):
    with pytest.raises(et.EtError) as e:
        et.et_stack_create(layers, M, dtype)
    return e.value.status


def test_create_validates_the_layer_chain():
    ok = et.et_stack_create([(8, 16, 1, 1, -1), (16, 8, 0, 1, 0)], 4, et.ET_F32)
    assert et.et_stack_workspace_bytes(ok) % 256 == 0
    assert _err([(8, 16, 0, 1, -1), (12, 8, 0, 1, -1)]) == et.ET_ERR_SHAPE          # widths do not chain
    assert _err([(8, 16, 0, 1, -1), (16, 4, 0, 1, 0)]) == et.ET_ERR_SHAPE           # residual width mismatch
    assert _err([(8, 15, 0, 2, -1)]) == et.ET_ERR_SHAPE                             # fold does not divide
    assert _err([(8, 16, 1, 2, -1)]) == et.ET_ERR_UNSUPPORTED                       # activation under a fold
    assert _err([(8, 16, 7, 1, -1)]) == et.ET_ERR_INVALID_ARG                       # unknown activation
    assert _err([(8, 16, 0, 1, 1)]) == et.ET_ERR_INVALID_ARG                        # residual from the future
    assert _err([(8, 16, 0, 1, -1)], M=0) == et.ET_ERR_INVALID_ARG
    assert _err([(8, 16, 0, 1, -1)], dtype=5) == et.ET_ERR_DTYPE
    assert _err([(8, 12, 0, 1, -1)], dtype=et.ET_BF16) == et.ET_ERR_UNSUPPORTED     # bf16 needs multiples of 8
    assert _err([(8, 384, 0, 3, -1)], dtype=et.ET_BF16) == et.ET_ERR_UNSUPPORTED    # folded width not a tile multiple


def test_calls_before_bind_are_refused():
    s = et.et_stack_create([(8, 16, 0, 1, -1)], 4, et.ET_F32)
    x = np.zeros(1, dtype=np.float32)     # any non-null address: nothing may be launched
    with pytest.raises(et.EtError) as e:
        et.et_forward_stack(s, x, x)
    assert e.value.status == et.ET_ERR_STATE
    with pytest.raises(et.EtError) as e:
        et.et_backward_elastic(s, x, np.zeros(2, dtype=np.uint8))
    assert e.value.status == et.ET_ERR_STATE
    with pytest.raises(et.EtError) as e:
        et.et_backward_elastic(s, x, np.zeros(3, dtype=np.uint8))                   # wrong mask length
    assert e.value.status == et.ET_ERR_INVALID_ARG


def test_workspace_is_sized_for_the_paper_shaped_stacks():
    w = wl.vit_b(params=False)
    s = et.et_stack_create(w.layers, w.M, et.ET_BF16)
    gb = et.et_stack_workspace_bytes(s) / 1e9
    assert 2.0 < gb < 20.0
    w = wl.vit_l(params=False)
    s = et.et_stack_create(w.layers, w.M, et.ET_BF16)
    assert et.et_stack_workspace_bytes(s) / 1e9 < 40.0


@pytest.mark.parametrize("variant", [et.ET_COST_STRICT, et.ET_COST_INCLUSIVE])
def test_time_selective_matches_oracle(variant):
    rng = np.random.default_rng(variant)
    for _ in range(100):
        n = int(rng.integers(1, 12))
        _, t_dw, t_dy = wl.selector_instance(rng, n, integer=False)
        mask = (rng.random(n) < 0.4).astype(np.uint8)
        assert et.et_time_selective(mask, t_dw, t_dy, variant) == pytest.approx(
            orc.t_selective(mask, t_dw, t_dy, variant), rel=1e-12, abs=1e-12)


@pytest.mark.parametrize("variant", [et.ET_COST_STRICT, et.ET_COST_INCLUSIVE])
def test_dp_matches_bruteforce(variant):
    rng = np.random.default_rng(100 + variant)
    for trial in range(120):
        n = int(rng.integers(1, 13))
        I, qw, qy = wl.selector_instance(rng, n, t_max=15)
        if trial % 4 == 0:
            I[rng.integers(0, n)] = -0.5
        if trial % 7 == 0:
            qw[rng.integers(0, n)] = 0
        qw, qy = qw.astype(np.int64), qy.astype(np.int64)
        budget = int(rng.integers(0, int(qw.sum() + qy.sum()) + 3))
        mask, val = et.et_select_dp_int(I, qw, qy, budget, variant)
        _, want = orc.select_bruteforce(I, qw, qy, budget, variant)
        assert abs(val - want) < 1e-12, (trial, n, budget)
        assert orc.t_selective(mask, qw, qy, variant) <= budget                     # returned mask is feasible
        assert abs(I[mask.astype(bool)].sum() - val) < 1e-12                        # and attains the value


def test_dp_larger_instance_against_depth_knapsack():
    rng = np.random.default_rng(5)
    I, qw, qy = wl.selector_instance(rng, 96, t_max=40)
    qw, qy = qw.astype(np.int64), qy.astype(np.int64)
    for frac in (0.1, 0.4, 0.8):
        budget = int(frac * (qw.sum() + qy.sum()))
        for variant in (et.ET_COST_STRICT, et.ET_COST_INCLUSIVE):
            mask, val = et.et_select_dp_int(I, qw, qy, budget, variant)
            assert abs(val - orc.select_by_depth_knapsack(I, qw, qy, budget, variant)) < 1e-9
            assert orc.t_selective(mask, qw, qy, variant) <= budget


def test_dp_edge_cases():
    I = np.array([0.5, 0.2, 0.9])
    w = np.array([3, 1, 2]); y = np.array([4, 0, 5])
    mask, val = et.et_select_dp_int(I, w, y, -1)
    assert not mask.any() and val == 0.0
    mask, val = et.et_select_dp_int(I, w, y, 0)
    assert not mask.any()
    mask, val = et.et_select_dp_int(I, w, y, 1000)
    assert mask.all() and abs(val - I.sum()) < 1e-12
    mask, val = et.et_select_dp_int(np.array([-1.0, -2.0]), np.array([1, 1]), np.array([1, 1]), 100)
    assert not mask.any() and val == 0.0                                             # empty selection is allowed
    mask, val = et.et_select_dp_int(np.zeros(0), np.zeros(0, dtype=np.int64), np.zeros(0, dtype=np.int64), 5)
    assert len(mask) == 0 and val == 0.0
    with pytest.raises(et.EtError):
        et.et_select_dp_int(I, np.array([-1, 0, 0]), y, 5)


def test_select_dp_quantised():
    rng = np.random.default_rng(9)
    for _ in range(30):
        n = int(rng.integers(2, 12))
        I, t_dw, t_dy = wl.selector_instance(rng, n, integer=False)
        rho = float(rng.uniform(0.2, 1.0))
        t_fwd = float(rng.uniform(0, 5))
        Tq = 200
        mask, val, est = et.et_select_dp(I, t_dw, t_dy, t_fwd, rho, Tq, et.ET_COST_STRICT)
        qw, qy, budget = orc.quantise(t_dw, t_dy, t_fwd, rho, Tq)
        _, want = orc.select_bruteforce(I, qw, qy, budget, orc.STRICT)
        assert abs(val - want) < 1e-9
        assert est == pytest.approx(orc.t_selective(mask, t_dw, t_dy, orc.STRICT), rel=1e-12, abs=1e-12)
        # flooring under-estimates each time by < 1 quantum: the true time overshoots the budget by < n quanta
        T = t_dw.sum() + t_dy.sum()
        assert est <= rho * (t_fwd + T) - t_fwd + 2 * n * T / Tq + 1e-9
    # rho = 1: everything is selected
    I, t_dw, t_dy = wl.selector_instance(rng, 40, integer=False)
    mask, val, est = et.et_select_dp(I + 0.01, t_dw, t_dy, 3.0, 1.0, 1000, et.ET_COST_INCLUSIVE)
    assert mask.all()


# ------------------------------------------------------------------ Section 6.3: pruning, threads, resolution
@pytest.mark.parametrize("variant", [et.ET_COST_STRICT, et.ET_COST_INCLUSIVE])
def test_pruned_and_threaded_dp_keep_the_optimum(variant):
    # skipping invalid and redundant subproblems, and sharing rows between threads, must not change the
    # value (Section 6.3: "without affecting optimality"); brute force is the referee
    rng = np.random.default_rng(300 + variant)
    for trial in range(80):
        n = int(rng.integers(1, 13))
        I, qw, qy = wl.selector_instance(rng, n, t_max=15)
        qw, qy = qw.astype(np.int64), qy.astype(np.int64)
        budget = int(rng.integers(0, int(qw.sum() + qy.sum()) + 3))
        _, want = orc.select_bruteforce(I, qw, qy, budget, variant)
        for prune in (True, False):
            for threads in (1, 3):
                mask, val, st = et.et_select_dp_int_ex(I, qw, qy, budget, variant, threads=threads, prune=prune)
                assert abs(val - want) < 1e-12, (trial, prune, threads)
                assert orc.t_selective(mask, qw, qy, variant) <= budget
                assert abs(I[mask.astype(bool)].sum() - val) < 1e-12


def test_dp_statistics_count_the_subproblems():
    # 4 tensors, unit weight-gradient times, error-gradient times 0, 3, 0, 5 (forward order), budget 6.
    # Counted from the output, tensor k costs at least low(k) = 1 + (error-gradient times above it):
    # 1, 6, 6, 9.  The budget reaches three of them, and of their rows 7-1, 7-6 and 7-6 entries can hold a
    # selection at all; no second tensor ever fits (every transition would start beyond t = 6).
    I = np.array([1.0, 1.0, 1.0, 1.0])
    w = np.array([1, 1, 1, 1], dtype=np.int64)
    y = np.array([0, 3, 0, 5], dtype=np.int64)
    mask, val, st = et.et_select_dp_int_ex(I, w, y, 6, et.ET_COST_STRICT)
    assert st["table_full"] == 4 * (12 + 1) and st["table_budget"] == 4 * 7
    assert st["rows_reached"] == 3 and st["visited"] == 6 + 1 + 1 and st["transitions"] == 0
    assert val == 1.0 and mask.sum() == 1
    _, _, full = et.et_select_dp_int_ex(I, w, y, 6, et.ET_COST_STRICT, prune=False)
    assert full["rows_reached"] == 4 and full["visited"] == 4 * 13
    assert full["transitions"] > st["transitions"]


def test_threaded_dp_on_a_large_instance():
    # N in the thousands: same value with 1 and 8 threads, and the same as the exact-cost knapsack route
    rng = np.random.default_rng(17)
    n = 1536
    I, t_dw, t_dy = wl.selector_instance(rng, n, integer=False)
    m1, v1, e1, s1 = et.et_select_dp_ex(I, t_dw, t_dy, 5.0, 0.4, 2000, et.ET_COST_STRICT, threads=1)
    m8, v8, e8, s8 = et.et_select_dp_ex(I, t_dw, t_dy, 5.0, 0.4, 2000, et.ET_COST_STRICT, threads=8)
    assert v1 == v8 and np.array_equal(m1, m8)
    assert s1["visited"] == s8["visited"] < s1["table_budget"] < s1["table_full"]
    assert s8["threads"] > 1 or (os.cpu_count() or 1) == 1      # rows this heavy are shared between threads
    qw, qy, budget = orc.quantise(t_dw, t_dy, 5.0, 0.4, 2000)
    assert abs(v1 - orc.select_by_depth_knapsack(I, qw, qy, budget, orc.STRICT)) < 1e-9


def test_resolution_sweep_converges():
    # Eq. 8: coarse resolutions blur the times; as T_q grows the selected value approaches the optimum of
    # the finest resolution and the over-run of the true budget (at most one quantum per tensor) vanishes
    rng = np.random.default_rng(23)
    I, t_dw, t_dy = wl.selector_instance(rng, 60, integer=False)
    T = t_dw.sum() + t_dy.sum()
    t_fwd, rho = 4.0, 0.5
    budget = rho * (t_fwd + T) - t_fwd
    overrun, value = [], []
    for Tq in (10, 100, 1000, 10000, 100000):
        mask, val, est, _ = et.et_select_dp_ex(I, t_dw, t_dy, t_fwd, rho, Tq)
        assert est <= budget + 2 * 60 * T / Tq + 1e-9
        overrun.append(max(0.0, est - budget) / budget)
        value.append(val)
    assert overrun[-1] < 1e-3 and overrun[-1] <= overrun[0] + 1e-12
    assert abs(value[-1] - value[-2]) <= 0.02 * value[-1]


# ------------------------------------------------------------------ options, guard words, no-allocation call (host side)
def test_stack_options_are_validated():
    s = et.et_stack_create([(8, 16, 0, 1, -1)], 4, et.ET_F32)
    et.et_stack_set_option(s, et.ET_OPTION_TWO_STREAMS, 0)
    et.et_stack_set_option(s, et.ET_OPTION_LAUNCH_OVERLAP, 0)
    et.et_stack_set_option(s, et.ET_OPTION_TILE_PLAN, et.ET_TILE_PLAN_SHARED)
    for opt, val in ((et.ET_OPTION_TWO_STREAMS, 2), (et.ET_OPTION_TILE_PLAN, 7), (99, 0)):
        with pytest.raises(et.EtError) as e:
            et.et_stack_set_option(s, opt, val)
        assert e.value.status == et.ET_ERR_INVALID_ARG


def test_guard_words_enlarge_the_workspace_and_need_a_bound_stack():
    layers = [(8, 16, 1, 1, -1), (16, 8, 0, 1, 0)]
    plain = et.et_stack_workspace_bytes(et.et_stack_create(layers, 4, et.ET_F32))
    et.et_debug_guard_regions(True)
    try:
        guarded = et.et_stack_create(layers, 4, et.ET_F32)
    finally:
        et.et_debug_guard_regions(False)
    extra = et.et_stack_workspace_bytes(guarded) - plain
    assert extra > 0 and extra % 256 == 0                          # 256 guard bytes after every region
    assert et.et_stack_workspace_bytes(et.et_stack_create(layers, 4, et.ET_F32)) == plain   # the switch is off again
    st, bad = et.et_debug_check_guards(guarded)
    assert st == et.ET_ERR_STATE and bad == -1                     # nothing bound yet: nothing to read


def test_create_refuses_more_rows_than_the_column_sum_grid_holds():
    assert _err([(8, 16, 0, 1, -1)], M=65535 * 128 + 1) == et.ET_ERR_UNSUPPORTED
    et.et_stack_create([(8, 16, 0, 1, -1)], 65535 * 128, et.ET_F32)


def test_noalloc_argument_checks_come_before_any_device_work():
    x = np.zeros(4, dtype=np.float32)        # any non-null address: refused calls dereference nothing
    for M, width, dtype, want in ((0, 8, et.ET_F32, et.ET_ERR_INVALID_ARG), (8, 8, 5, et.ET_ERR_DTYPE),
                                  (128 * (et.ET_NOALLOC_SCRATCH_FLOATS // 4096) + 1, 4096, et.ET_F32, et.ET_ERR_TOO_LARGE),
                                  (65535 * 128 + 1, 8, et.ET_F32, et.ET_ERR_TOO_LARGE)):
        with pytest.raises(et.EtError) as e:
            et.et_bias_grad_noalloc(x, M, width, dtype, x)
        assert e.value.status == want, (M, width)
