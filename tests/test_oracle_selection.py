"""Pins of the oracle's integer parts: which work a mask executes (the paper's two
worked examples), the time model, and the selector optimum by two independent routes."""
import json
import os

import numpy as np
import pytest

import workloads as wl
from oracle import elastic_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def test_time_model_example_section_2_2():
    g = _gold("time_model_section_2_2.json")
    L = g["n_layers"]
    mask = np.zeros(2 * L, dtype=np.uint8)
    for l1 in g["selected_layers_1based"]:
        mask[2 * (l1 - 1)] = 1                     # its kernel
    plan = orc.exec_plan(L, mask)
    assert [l + 1 for l in range(L) if plan.wgrad[l]] == g["paid_t_dw_1based"]
    assert [l + 1 for l in range(L) if plan.dgrad[l]] == g["paid_t_dy_1based"]
    assert plan.deepest == 2 and not plan.bgrad.any()
    # the same through the cost model, with distinct powers of two as times
    t_dw = np.array([2.0 ** l for l in range(L)])
    t_dy = np.array([2.0 ** (8 + l) for l in range(L)])
    layer_mask = np.array([0, 0, 1, 0, 0])
    assert orc.t_selective(layer_mask, t_dw, t_dy, orc.STRICT) == t_dw[2] + t_dy[3] + t_dy[4]


def test_f_mask_example_eq_3():
    g = _gold("f_mask_eq_3.json")
    assert orc.f_mask(g["M"]).tolist() == g["f_of_M"]
    t_dw = np.arange(1.0, 8.0)
    t_dy = 10.0 * np.arange(1.0, 8.0)
    assert orc.t_selective(g["M"], t_dw, t_dy, orc.INCLUSIVE) == 4 + 5 + 10 * (4 + 5 + 6 + 7)
    assert orc.t_selective(g["M"], t_dw, t_dy, orc.STRICT) == 4 + 5 + 10 * (5 + 6 + 7)


def test_exec_plan_cases():
    L = 4
    # nothing selected: nothing runs
    p = orc.exec_plan(L, np.zeros(8, dtype=np.uint8))
    assert p.deepest == L and not (p.dgrad.any() or p.wgrad.any() or p.bgrad.any() or p.updated.any())
    # only a bias of layer 1: layers 2, 3 pass gradients, no kernel gradient anywhere
    m = np.zeros(8, dtype=np.uint8); m[3] = 1
    p = orc.exec_plan(L, m)
    assert p.deepest == 1 and p.dgrad.tolist() == [False, False, True, True]
    assert not p.wgrad.any() and p.bgrad.tolist() == [False, True, False, False]
    # everything selected = full backprop: every layer but the first passes a gradient
    p = orc.exec_plan(L, np.ones(8, dtype=np.uint8))
    assert p.deepest == 0 and p.dgrad.tolist() == [False, True, True, True] and p.wgrad.all() and p.bgrad.all()
    # the tiny-MLP workload's mask: layer 2 only => dgrad(3), wgrad(2), bgrad(2)
    w = wl.tiny_mlp(params=False)
    p = orc.exec_plan(w.L, w.mask)
    assert p.deepest == 2 and p.dgrad.tolist() == [False, False, False, True]
    assert p.wgrad.tolist() == [False, False, True, False] and p.bgrad.tolist() == p.wgrad.tolist()
    fl = orc.executed_flops(w.layers, w.M, p)
    assert fl == 2.0 * 256 * 128 * 512 + 2.0 * 256 * 512 * 128


def test_increment_eq_7():
    # adding tensor k (counted from the output side) to a solution whose closest
    # selected tensor is k_c costs t_dw(k) + sum_{j=k_c}^{k-1} t_dy(j)
    rng = np.random.default_rng(0)
    n = 9
    _, t_dw, t_dy = wl.selector_instance(rng, n)
    t_dy = rng.integers(1, 20, size=n).astype(float)
    for _ in range(50):
        m_out = (rng.random(n) < 0.4)                       # index 0 = last tensor (output side)
        if not m_out.any():
            continue
        kc = int(np.max(np.nonzero(m_out)[0]))
        if kc == n - 1:
            continue
        k = int(rng.integers(kc + 1, n))
        m2 = m_out.copy(); m2[k] = True
        fw = lambda m: m[::-1].astype(np.uint8)            # to forward order
        before = orc.t_selective(fw(m_out), t_dw[::-1], t_dy[::-1], orc.STRICT)
        after = orc.t_selective(fw(m2), t_dw[::-1], t_dy[::-1], orc.STRICT)
        assert after - before == t_dw[k] + t_dy[kc:k].sum()


@pytest.mark.parametrize("variant", [orc.STRICT, orc.INCLUSIVE])
def test_bruteforce_matches_depth_knapsack(variant):
    rng = np.random.default_rng(7 + variant)
    for trial in range(40):
        n = int(rng.integers(1, 11))
        I, qw, qy = wl.selector_instance(rng, n, t_max=12)
        if trial % 5 == 0:
            I[rng.integers(0, n)] = -0.3                   # a harmful tensor is never worth selecting
        qw, qy = qw.astype(np.int64), qy.astype(np.int64)
        budget = int(rng.integers(0, int(qw.sum() + qy.sum()) + 2))
        mask, val = orc.select_bruteforce(I, qw, qy, budget, variant)
        assert orc.t_selective(mask, qw, qy, variant) <= budget
        assert abs(I[mask.astype(bool)].sum() - val) < 1e-12
        assert abs(orc.select_by_depth_knapsack(I, qw, qy, budget, variant) - val) < 1e-12


def test_budget_of_full_time_selects_everything():
    # rho = 100 %: every tensor is affordable (Section 3), also after flooring (Eq. 8)
    rng = np.random.default_rng(3)
    I, t_dw, t_dy = wl.selector_instance(rng, 10, integer=False)
    I = I + 0.01
    qw, qy, budget = orc.quantise(t_dw, t_dy, t_fwd=3.0, rho=1.0, Tq=50)
    assert qw.sum() + qy.sum() <= budget
    mask, val = orc.select_bruteforce(I, qw, qy, budget, orc.INCLUSIVE)
    assert mask.all() and abs(val - I.sum()) < 1e-12


def test_quantise_eq_8():
    qw, qy, budget = orc.quantise([1.0, 2.5, 0.49], [0.5, 0.0, 0.51], t_fwd=0.0, rho=0.5, Tq=10)
    # T = 5, Z = 2
    assert qw.tolist() == [2, 5, 0] and qy.tolist() == [1, 0, 1] and budget == 5


@pytest.mark.parametrize("variant", [orc.STRICT, orc.INCLUSIVE])
def test_knapsack_mask_matches_bruteforce(variant):
    rng = np.random.default_rng(40 + variant)
    for trial in range(40):
        n = int(rng.integers(1, 11))
        I, qw, qy = wl.selector_instance(rng, n, t_max=12)
        if trial % 3 == 0:
            I[rng.integers(0, n)] = -0.2
        qw, qy = qw.astype(np.int64), qy.astype(np.int64)
        budget = int(rng.integers(0, int(qw.sum() + qy.sum()) + 2))
        mask, val = orc.select_depth_knapsack_mask(I, qw, qy, budget, variant)
        _, want = orc.select_bruteforce(I, qw, qy, budget, variant)
        assert abs(val - want) < 1e-12
        assert orc.t_selective(mask, qw, qy, variant) <= budget
        assert abs(I[mask.astype(bool)].sum() - val) < 1e-12


def test_train_schedule_structure_and_progress():
    layers = wl.vit_blocks(2, 8, 16)
    w = wl.small_stack(layers, 12, wl.DT_F32, 3, w_std=0.3)
    L = len(layers)
    t_dw = np.array([2.0 * ly.in_features * ly.out_features if t % 2 == 0 else ly.out_features
                     for ly in layers for t in range(2)])
    t_dy = np.array([2.0 * ly.in_features * ly.out_features if t % 2 == 0 else 0.0
                     for ly in layers for t in range(2)])
    out = orc.train_schedule(w.layers, w.W, w.b, w.x, w.target, lr=0.05, steps=24, period=8, window=3,
                             rho=0.4, t_dw=t_dw, t_dy=t_dy, Tq=200)
    assert out["losses"][-1] < out["losses"][0]
    assert len(out["importances"]) == 3
    for step, m in enumerate(out["masks"]):
        if step % 8 < 3:
            assert m.all()                                   # every tensor trains during the window
        else:
            assert not m.all()                               # rho = 0.4 cannot afford everything
            assert orc.t_selective(m, t_dw, t_dy) <= 0.4 * (t_dw.sum() + t_dy.sum()) * 1.05
            if step % 8 > 3:
                assert np.array_equal(m, out["masks"][step - 1])   # masks only change at a reselection
    # importances of useful updates are negative sums (the loss went down along them)
    assert (np.concatenate(out["importances"]) <= 1e-12).mean() > 0.8
