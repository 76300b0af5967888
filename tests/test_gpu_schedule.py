"""The elastic training schedule (all-tensor window, importance evaluation with the weight
change since the window start, re-selection, masked steps) on the GPU against the oracle's
own run of the same schedule, and the selector fed with measured per-tensor times."""
import numpy as np
import pytest
import torch

import paper_2312_14227_b200 as et
from paper_2312_14227_b200.elastic_loop import ElasticLoop
from workloads import flop_costs
import workloads as wl
from oracle import elastic_oracle as orc

pytestmark = pytest.mark.gpu


def test_schedule_fp32_reduced_twin_matches_oracle_trajectory():
    import gpu_harness as h
    # reduced twin of the ViT-L schedule: same wiring and schedule logic, small widths, fp32 storage
    # (bf16 storage cannot hold updates of lr * g next to weights of 0.02 without master weights)
    layers = wl.vit_blocks(8, 64, 256)
    w = wl.small_stack(layers, 197, wl.DT_F32, 17, w_std=0.02)
    steps, period, window, rho, Tq = 90, 30, 6, 0.4, 300
    t_dw, t_dy = flop_costs(w.layers, w.M)
    ref = orc.train_schedule(w.layers, w.W, w.b, w.x, w.target, w.lr, steps, period, window, rho, t_dw, t_dy, Tq=Tq)

    run = h.GpuRun(w)
    loop = ElasticLoop(run.stack, run.W, run.b, run.x, run.target, w.lr, period, window, rho, t_dw, t_dy, Tq=Tq)
    got = loop.run(steps)
    assert et.et_device_status(run.stack) == et.ET_OK

    assert len(got["importances"]) == len(ref["importances"]) == 3
    qw, qy, budget = orc.quantise(t_dw, t_dy, 0.0, rho, Tq)
    for S_gpu, S_ref in zip(got["importances"], ref["importances"]):
        assert np.abs(S_gpu - S_ref).max() <= 2e-3 * np.abs(S_ref).max()
    for step in range(steps):
        m_gpu, m_ref = got["masks"][step], ref["masks"][step]
        if not np.array_equal(m_gpu, m_ref):
            # equal-value optima may differ; both must be feasible and equally good on the oracle's importances
            k = step // period
            I = -ref["importances"][k]
            assert orc.t_selective(m_gpu, qw, qy) <= budget
            assert abs(I[m_gpu.astype(bool)].sum() - I[m_ref.astype(bool)].sum()) <= 1e-3 * abs(I[m_ref.astype(bool)].sum())
    np.testing.assert_allclose(got["losses"], ref["losses"], rtol=2e-3)
    assert got["losses"][-1] < got["losses"][0]
    # tensors frozen through a masked phase did not move during it: compare with the oracle's final weights
    final = orc.tensors_of(ref["W"], ref["b"])
    for t, p in enumerate(run.params()):
        assert np.abs(h.to_np(p) - final[t]).max() <= 1e-3


def test_schedule_bf16_with_master_weights_follows_oracle():
    import gpu_harness as h
    # bf16 storage and tensor-core kernels, fp32 master weights: the schedule still follows the
    # float64 run closely (without master weights most updates would be rounded away)
    layers = wl.vit_blocks(4, 256, 512)
    w = wl.small_stack(layers, 394, wl.DT_BF16, 23, w_std=0.02)
    steps, period, window, rho, Tq = 60, 30, 6, 0.5, 300
    t_dw, t_dy = flop_costs(w.layers, w.M)
    ref = orc.train_schedule(w.layers, w.W, w.b, w.x, w.target, w.lr, steps, period, window, rho, t_dw, t_dy, Tq=Tq)
    run = h.GpuRun(w)
    loop = ElasticLoop(run.stack, run.W, run.b, run.x, run.target, w.lr, period, window, rho, t_dw, t_dy, Tq=Tq,
                       master=True)
    got = loop.run(steps)
    assert et.et_device_status(run.stack) == et.ET_OK
    np.testing.assert_allclose(got["losses"], ref["losses"], rtol=2e-2)
    assert got["losses"][-1] < got["losses"][0]
    for S_gpu, S_ref in zip(got["importances"], ref["importances"]):
        assert np.abs(S_gpu - S_ref).max() <= 5e-2 * np.abs(S_ref).max()
    final = orc.tensors_of(ref["W"], ref["b"])
    for t, p in enumerate(loop.master):
        assert np.abs(h.to_np(p) - final[t]).max() <= 2e-3
    # the bf16 tensors are the roundings of their masters
    for p16, p32 in zip(run.params(), loop.master):
        assert torch.equal(p16, p32.to(torch.bfloat16))


def test_selector_on_measured_costs_bf16():
    import gpu_harness as h
    # per-tensor times measured with CUDA events, seeded Uniform(0,1) importances, budgets as a
    # fraction of the full backward time (no forward term): the selected masks run, match the
    # oracle, and the measured step time follows the model's estimate
    w = wl.vit_b(seed=5, n_blocks=3, tokens=4096, name="vit_b_3blocks")
    run = h.GpuRun(w)
    run.forward_loss()
    t_dw, t_dy, t_fwd = et.et_profile_costs(run.stack, run.x, run.y, run.dY, iters=10)
    assert t_fwd > 0 and (t_dy[1::2] == 0).all() and t_dy[0] == 0 and (t_dw > 0).all() and (t_dy[2::2] > 0).all()
    rng = np.random.default_rng(9)
    I = rng.random(2 * w.L)
    total = t_dw.sum() + t_dy.sum()
    prev = -1
    for rho in (0.25, 0.5, 1.0):
        mask, val, est = et.et_select_dp(I, t_dw, t_dy, 0.0, rho, 1000, et.ET_COST_STRICT)
        assert est <= rho * total * 1.03
        assert mask.sum() >= prev
        prev = mask.sum()
        if rho == 1.0:
            assert mask.all()
        if mask.any():
            w.mask = mask
            h.check_step(w, mask, 2e-2)


def _trainable(layers):
    return np.array([0 if ly.kind in (wl.KIND_ATTENTION, wl.KIND_IM2COL) else 1 for ly in layers for _ in (0, 1)], dtype=bool)


def test_schedule_with_normalisation_layers_fp32_matches_oracle_trajectory():
    import gpu_harness as h
    # the pre-norm twin: gamma and beta take part in the selection like any other tensor
    layers = wl.vit_blocks_prenorm(4, 64, 256)
    w = wl.small_stack(layers, 197, wl.DT_F32, 18, w_std=0.05)
    steps, period, window, rho, Tq = 60, 30, 6, 0.4, 300
    t_dw, t_dy = flop_costs(w.layers, w.M)
    ref = orc.train_schedule(w.layers, w.W, w.b, w.x, w.target, w.lr, steps, period, window, rho, t_dw, t_dy, Tq=Tq)
    run = h.GpuRun(w)
    loop = ElasticLoop(run.stack, run.W, run.b, run.x, run.target, w.lr, period, window, rho, t_dw, t_dy, Tq=Tq)
    got = loop.run(steps)
    assert et.et_device_status(run.stack) == et.ET_OK
    for S_gpu, S_ref in zip(got["importances"], ref["importances"]):
        assert np.abs(S_gpu - S_ref).max() <= 2e-3 * np.abs(S_ref).max()
    np.testing.assert_allclose(got["losses"], ref["losses"], rtol=2e-3)
    assert got["losses"][-1] < got["losses"][0]
    qw, qy, budget = orc.quantise(t_dw, t_dy, 0.0, rho, Tq)
    for step in range(steps):
        m_gpu, m_ref = got["masks"][step], ref["masks"][step]
        if not np.array_equal(m_gpu, m_ref):
            I = -ref["importances"][step // period]
            assert orc.t_selective(m_gpu, qw, qy) <= budget
            assert abs(I[m_gpu.astype(bool)].sum() - I[m_ref.astype(bool)].sum()) <= 1e-3 * abs(I[m_ref.astype(bool)].sum())
    final = orc.tensors_of(ref["W"], ref["b"])
    for t, p in enumerate(run.params()):
        assert np.abs(h.to_np(p) - final[t]).max() <= 1e-3


def test_schedule_full_transformer_blocks_bf16_with_master_weights():
    import gpu_harness as h
    # normalisation layers and the attention core in the stack; layers without tensors never enter a mask
    layers = wl.vit_blocks_full(2, 128, 256, heads=2, seq=49)
    w = wl.small_stack(layers, 8 * 49, wl.DT_BF16, 24, w_std=0.05)
    live = _trainable(layers)
    steps, period, window, rho, Tq = 60, 30, 6, 0.5, 300
    t_dw, t_dy = flop_costs(w.layers, w.M)
    ref = orc.train_schedule(w.layers, w.W, w.b, w.x, w.target, w.lr, steps, period, window, rho, t_dw, t_dy, Tq=Tq)
    run = h.GpuRun(w)
    loop = ElasticLoop(run.stack, run.W, run.b, run.x, run.target, w.lr, period, window, rho, t_dw, t_dy, Tq=Tq,
                       master=True)
    got = loop.run(steps)
    assert et.et_device_status(run.stack) == et.ET_OK
    assert all(not m[~live].any() for m in got["masks"])
    np.testing.assert_allclose(got["losses"], ref["losses"], rtol=2e-2)
    assert got["losses"][-1] < got["losses"][0]
    for S_gpu, S_ref in zip(got["importances"], ref["importances"]):
        assert np.abs(S_gpu - S_ref)[live].max() <= 5e-2 * np.abs(S_ref).max()
    final = orc.tensors_of(ref["W"], ref["b"])
    for t, p in enumerate(loop.master):
        if live[t]:
            assert np.abs(h.to_np(p) - final[t]).max() <= 2e-3
