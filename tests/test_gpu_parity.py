"""Parity of the CUDA path against the float64 oracle, through the C ABI.
Bars: executed-work sets and frozen weights exact; gradients / importances within 1e-4
(fp32 stacks) or 2e-2 (bf16 stacks) max-norm relative error; updated weights within 1e-3."""
import numpy as np
import pytest
import torch

import paper_2312_14227_b200 as et
import workloads as wl
from oracle import elastic_oracle as orc

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 2e-2


def _h():
    import gpu_harness
    return gpu_harness


def test_tiny_mlp_fp32_config():
    h = _h()
    w = wl.tiny_mlp()
    rep = h.check_step(w, w.mask, TOL_F32)
    assert rep.deepest == 2 and rep.dgrad.tolist() == [0, 0, 0, 1]
    assert rep.wgrad.tolist() == [0, 0, 1, 0] and rep.bgrad.tolist() == [0, 0, 1, 0]


def test_tiny_mlp_fp32_all_selected_is_full_backprop():
    h = _h()
    w = wl.tiny_mlp()
    h.check_step(w, np.ones(2 * w.L, dtype=np.uint8), TOL_F32)


def test_importance_of_a_gradient_step_fp32_and_bf16():
    # dw proportional to -g (Eq. 2 with the update a gradient step makes): plain relative error
    h = _h()
    w = wl.tiny_mlp()
    h.check_step(w, np.ones(2 * w.L, dtype=np.uint8), TOL_F32, aligned_delta=True)
    w = wl.vit_b(seed=12, p_select=0.5, n_blocks=2, tokens=520, d=256, ffn=768)
    w.mask[:] = 1
    h.check_step(w, w.mask, TOL_BF16, aligned_delta=True)
    # the same through the snapshot form of the call (dw = W - snapshot formed on the fly)
    c = h.StepChecker(w, TOL_BF16)
    c.check(w.mask, aligned_delta=True, snapshot=True)
    c.check(w.mask, snapshot=True)


def _all_kinds_layers(scale=1):
    s = scale
    return [
        wl.Layer(6 * s, 9 * s, fold=3),
        wl.Layer(3 * s, 6 * s, residual_src=0),
        wl.Layer(6 * s, 10 * s, act=wl.ACT_GELU_TANH),
        wl.Layer(10 * s, 6 * s, residual_src=2),
        wl.Layer(6 * s, 5 * s, act=wl.ACT_RELU),
        wl.Layer(5 * s, 6 * s, act=wl.ACT_GELU_TANH, residual_src=4),
        wl.Layer(6 * s, 4 * s),
    ]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_fp32_ragged_all_layer_kinds(seed):
    h = _h()
    rng = np.random.default_rng(seed)
    layers = _all_kinds_layers(scale=[1, 11, 23][seed])          # widths not multiples of any tile
    M = [7, 131, 77][seed]
    for trial in range(3):
        mask = (rng.random(2 * len(layers)) < 0.4).astype(np.uint8)
        w = wl.small_stack(layers, M, wl.DT_F32, seed * 10 + trial, mask=mask, w_std=0.2, bias_std=0.1)
        h.check_step(w, mask, TOL_F32)


def test_empty_mask_launches_nothing():
    h = _h()
    w = wl.tiny_mlp()
    run = h.GpuRun(w)
    run.forward_loss()
    before = [p.clone() for p in run.params()]
    delta = [h.to_dev(d, w.dtype) for d in wl.draw_delta(w, 1)]
    n0 = et.et_launch_count()
    rep = run.backward(np.zeros(2 * w.L, dtype=np.uint8), None, delta, flags=et.ET_FLAG_FUSE_SGD, lr=0.1)
    assert et.et_launch_count() == n0 and rep.launches == 0 and rep.deepest == w.L
    assert rep.flops_executed == 0.0 and not rep.dgrad.any()
    assert torch.all(run.importance == 0)
    for p, q in zip(run.params(), before):
        assert torch.equal(p, q)


def test_backward_before_forward_is_refused():
    h = _h()
    w = wl.tiny_mlp()
    run = h.GpuRun(w)
    with pytest.raises(et.EtError) as e:
        et.et_backward_elastic(run.stack, run.dY, w.mask)
    assert e.value.status == et.ET_ERR_STATE


def test_standalone_importance_and_sgd_match_fused_path():
    h = _h()
    w = wl.tiny_mlp()
    mask = np.ones(2 * w.L, dtype=np.uint8); mask[2] = 0; mask[7] = 0
    delta_np = wl.draw_delta(w, 3)
    ref = h.oracle_step(w, mask, delta_np)
    run = h.GpuRun(w)
    run.forward_loss()
    before = [p.clone() for p in run.params()]
    grads = run.alloc_grads(mask)
    run.backward(mask, grads, None)                       # gradients only
    delta = [h.to_dev(d, w.dtype) for d in delta_np]
    imp = torch.full((2 * w.L,), float("nan"), dtype=torch.float32, device=h.DEV)
    et.et_importance(run.stack, mask, grads, delta, imp)
    et.et_sgd_masked(run.stack, mask, grads, w.lr)
    imp = h.to_np(imp)
    for t in range(2 * w.L):
        if mask[t]:
            assert h.importance_err(imp[t], ref["grads"][t], delta_np[t]) <= TOL_F32
            assert np.abs(h.to_np(run.params()[t]) - ref["new"][t]).max() <= 1e-3
        else:
            assert imp[t] == 0.0 and torch.equal(run.params()[t], before[t])


# ------------------------------------------------------------------ bf16 / tensor-core path
def test_bf16_small_vit_block_ragged_rows():
    h = _h()
    # one transformer-shaped block, widths = one to three tiles, rows not a multiple of 128 or 64
    w = wl.vit_b(seed=11, p_select=0.6, n_blocks=2, tokens=300, d=256, ffn=512, name="vit_small")
    w.mask[:] = 1
    h.check_step(w, w.mask, TOL_BF16)


@pytest.mark.parametrize("gemm_list", [True, False])
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_bf16_random_masks_small_vit(seed, gemm_list):
    """Both launch schemes of the backward pass: every GEMM of the call in one cooperative launch
    (gemm_list) and one launch per GEMM on two streams."""
    h = _h()
    w = wl.vit_b(seed=20 + seed, p_select=0.3, n_blocks=3, tokens=[197, 520, 1000, 333][seed], d=256, ffn=768)
    if not w.mask.any():
        w.mask[-2:] = 1
    rep = h.check_step(w, w.mask, TOL_BF16, gemm_list=gemm_list)
    n_gemms = int(rep.dgrad.sum() + rep.wgrad.sum())
    if gemm_list:
        assert rep.launches <= 6                     # loss-side kernels, one GEMM launch, two grouped finishers
    else:
        assert rep.launches >= n_gemms


def test_bf16_one_launch_backward_all_masks_of_a_block():
    """Every selection of the eight tensors of one transformer block (256 masks) through the one-launch
    backward: the task list, its dependency counters and the fused weight-gradient epilogues are rebuilt
    for each mask on the same stack."""
    h = _h()
    w = wl.vit_b(seed=41, p_select=0.5, n_blocks=1, tokens=600, d=256, ffn=512)
    c = h.StepChecker(w, TOL_BF16, gemm_list=True)
    for bits in range(1, 256, 7):
        mask = np.array([(bits >> i) & 1 for i in range(8)], dtype=np.uint8)
        c.check(mask)
    c.check(np.ones(8, dtype=np.uint8), aligned_delta=True)
    c.check(np.ones(8, dtype=np.uint8), snapshot=True)


def test_bf16_ragged_widths_and_bias_only_selection():
    h = _h()
    layers = [wl.Layer(72, 200, act=wl.ACT_RELU), wl.Layer(200, 72, residual_src=0),
              wl.Layer(72, 328, act=wl.ACT_GELU_TANH), wl.Layer(328, 136)]
    mask = np.array([0, 1, 0, 0, 1, 0, 0, 1], dtype=np.uint8)
    w = wl.small_stack(layers, 450, wl.DT_BF16, 5, mask=mask, w_std=0.1, bias_std=0.05)
    h.check_step(w, mask, TOL_BF16)
    w = wl.small_stack(layers, 129, wl.DT_BF16, 6, mask=np.ones(8, dtype=np.uint8), w_std=0.1, bias_std=0.05)
    h.check_step(w, w.mask, TOL_BF16)


def test_bf16_fewer_rows_than_one_tile():
    # 40 rows: every TMA box is taller than the tensors, half of each CTA pair works on padding
    h = _h()
    layers = [wl.Layer(64, 128, act=wl.ACT_GELU_TANH), wl.Layer(128, 64, residual_src=0), wl.Layer(64, 256, fold=1)]
    w = wl.small_stack(layers, 40, wl.DT_BF16, 8, mask=np.ones(6, dtype=np.uint8), w_std=0.1, bias_std=0.05)
    h.check_step(w, w.mask, TOL_BF16)


def test_bf16_resnet_1x1_config():
    h = _h()
    w = wl.resnet_1x1()
    # He-initialised weights reach 0.5 and gradients reach 35 here: a bf16 store alone is
    # off by up to 2^-9 |w| ~ 1e-3, so the weight bound is the derived one
    c = h.StepChecker(w, TOL_BF16)
    stats = {}
    c.check(w.mask, derived_w_tol=True, stats=stats)
    # Eq. 2 with the update a gradient step makes (dw = -c g): plain relative error of every importance
    c.check(w.mask, derived_w_tol=True, stats=stats, aligned_delta=True)
    print("resnet_1x1 parity diagnostics", stats)


def test_bf16_deterministic():
    h = _h()
    w = wl.vit_b(seed=31, p_select=0.5, n_blocks=2, tokens=700, d=256, ffn=512)
    w.mask[:] = 1
    outs = []
    for _ in range(2):
        run = h.GpuRun(w)
        run.forward_loss()
        grads = run.alloc_grads(w.mask)
        delta = [h.to_dev(d, w.dtype) for d in wl.draw_delta(w, 4)]
        run.backward(w.mask, grads, delta)
        outs.append(([g.clone() for g in grads], run.importance.clone()))
    for a, b in zip(outs[0][0], outs[1][0]):
        assert torch.equal(a, b)
    assert torch.equal(outs[0][1], outs[1][1])


@pytest.fixture(scope="module")
def vit_b_checker():
    """The benchmark configuration (12 blocks, 12608 tokens) bound once: the oracle's forward pass of
    the whole stack takes about half a minute and does not depend on the mask."""
    c = _h().StepChecker(wl.vit_b(), TOL_BF16)
    yield c
    del c
    torch.cuda.empty_cache()


def test_bf16_vit_b_full_size_config(vit_b_checker):
    """The benchmark configuration itself (12 blocks, 12608 tokens, Bernoulli(0.3) mask),
    launched exactly as bench.py launches it, against the full oracle; the importances both for a
    random dw (bound relative to ||g||_inf ||dw||_2) and for dw = -c g (plain relative error)."""
    c = vit_b_checker
    stats = {}
    c.check(c.w.mask, stats=stats)
    c.check(c.w.mask, stats=stats, aligned_delta=True)
    # the same step launched GEMM by GEMM on two streams (the path stacks with other layer kinds take)
    et.et_stack_set_option(c.run.stack, et.ET_OPTION_GEMM_LIST, 0)
    c.check(c.w.mask, stats=stats)
    et.et_stack_set_option(c.run.stack, et.ET_OPTION_GEMM_LIST, 1)
    print("vit_b parity diagnostics", stats)


def test_bf16_vit_b_full_size_selector_masks(vit_b_checker):
    """Masks chosen by the host selector (Section 6, Eq. 3) at time budgets rho of the full backward
    pass on per-tensor times measured on this stack, seeded Uniform(0,1) importances, T_fwd = 0,
    T_q = 1000: every mask runs at full size and matches the oracle."""
    c = vit_b_checker
    run, w = c.run, c.w
    c._restore()         # the profiler re-runs the forward pass: it must see the weights the oracle has,
                         # not the ones the previous check's fused update left behind
    t_dw, t_dy, t_fwd = et.et_profile_costs(run.stack, run.x, run.y, run.dY, iters=5)
    run.forward_loss()
    assert t_fwd > 0 and (t_dy[1::2] == 0).all() and t_dy[0] == 0 and (t_dw > 0).all() and (t_dy[2::2] > 0).all()
    I = np.random.default_rng(9).random(2 * w.L)
    total = t_dw.sum() + t_dy.sum()
    prev, stats = -1, {}
    for rho in (0.25, 0.5, 1.0):
        mask, val, est = et.et_select_dp(I, t_dw, t_dy, 0.0, rho, 1000, et.ET_COST_STRICT)
        # Eq. 8 floors every time to a multiple of total / T_q, so each term the selector adds up may be
        # under-estimated by less than one quantum: the true time of a feasible mask exceeds the budget by
        # at most one quantum per selected tensor (t_dw) plus one per layer above the deepest (t_dy)
        deepest = int(np.flatnonzero(mask)[0]) // 2
        terms = int(mask.sum()) + (w.L - 1 - deepest)
        assert est <= rho * total + terms * total / 1000
        assert mask.sum() >= prev
        prev = int(mask.sum())
        if rho == 1.0:
            assert mask.all()
        assert mask.any()
        rep = c.check(mask, stats=stats)
        print(f"rho={rho}: {prev} tensors, deepest layer {rep.deepest}, estimated {est:.3f} ms of {total:.3f} ms")
    print("vit_b selector-mask parity diagnostics", stats)


def test_bf16_vit_l_shapes_snapshot_importance_and_master_weights():
    """The shapes of the elastic-schedule configuration (d = 1024, FFN 4096, QKV 3072, 6304 tokens; 4 of
    its 24 blocks: tile plans depend on widths and rows, not on depth), driven the way the schedule
    drives them: fp32 master weights, importances from the weight change since a snapshot (Section 3.1).
    One all-tensor step as in the window, one step with a selector mask at rho = 0.4."""
    h = _h()
    full = wl.vit_l(params=False)
    w = wl.vit_l(n_blocks=4)
    assert w.M == full.M and [(l.in_features, l.out_features) for l in w.layers] == \
        [(l.in_features, l.out_features) for l in full.layers[:w.L]]
    c = h.StepChecker(w, TOL_BF16, master=True)
    stats = {}
    ones = np.ones(2 * w.L, dtype=np.uint8)
    c.check(ones, snapshot=True, stats=stats)
    c.check(ones, snapshot=True, aligned_delta=True, stats=stats)
    t_dw, t_dy = wl.flop_costs(w.layers, w.M)
    I = np.random.default_rng(10).random(2 * w.L)
    mask, _, _ = et.et_select_dp(I, t_dw, t_dy, 0.0, 0.4, 1000, et.ET_COST_STRICT)
    assert mask.any() and not mask.all()
    c.check(mask, snapshot=True, stats=stats)
    print("vit_l-shape parity diagnostics", stats)


def test_device_status_reports_a_recorded_timeout():
    # every bounded device-side wait that gives up leaves a code in the status word at the start
    # of the workspace; the host turns it into ET_ERR_TIMEOUT.  The word is planted from the host
    # here: nothing on the GPU is made to wait.
    h = _h()
    w = wl.tiny_mlp()
    run = h.GpuRun(w)
    assert et.et_device_status(run.stack) == et.ET_OK
    run.ws[:4] = torch.tensor([2, 0, 0, 0], dtype=torch.uint8, device=h.DEV)
    assert et.et_device_status(run.stack) == et.ET_ERR_TIMEOUT
    run.ws[:4] = 0
    assert et.et_device_status(run.stack) == et.ET_OK


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, TOL_F32), (wl.DT_BF16, TOL_BF16)])
def test_ablation_metrics_weight_and_gradient_magnitude(dtype, tol):
    # the two non-additive metrics of the paper's ablation, as stand-alone reductions
    h = _h()
    layers = [wl.Layer(72, 200, act=wl.ACT_RELU), wl.norm_layer(200), wl.Layer(200, 136)]
    mask = np.array([1, 1, 1, 0, 1, 1], dtype=np.uint8)
    w = wl.small_stack(layers, 300, dtype, 71, mask=mask, w_std=0.1, bias_std=0.05)
    run = h.GpuRun(w)
    run.forward_loss()
    grads = run.alloc_grads(mask)
    run.backward(mask, grads, None)
    out = torch.full((6,), float("nan"), dtype=torch.float32, device=h.DEV)
    et.et_tensor_metric(run.stack, mask, et.ET_METRIC_WEIGHT_MAGNITUDE, None, out)
    want = orc.magnitude_metric(orc.tensors_of(w.W, w.b), mask)
    got = h.to_np(out)
    assert got[3] == 0.0 and np.all(np.abs(got - want) <= 1e-5 * np.abs(want) + 1e-12)      # inputs are exact in both
    et.et_tensor_metric(run.stack, mask, et.ET_METRIC_GRADIENT_MAGNITUDE, grads, out)
    ref = h.oracle_step(w, mask)
    want = orc.magnitude_metric([ref["grads"].get(t) if mask[t] else None for t in range(6)], mask)
    got = h.to_np(out)
    assert got[3] == 0.0 and np.all(np.abs(got - want) <= tol * np.abs(want) + 1e-12)
