"""Parity of the attention core as a stack member (a layer without trainable tensors) against the
float64 oracle, through the C ABI.  bf16 stacks only; same bars as the other bf16 parity tests."""
import numpy as np
import pytest

import paper_2312_14227_b200 as et
import workloads as wl

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def _h():
    import gpu_harness
    return gpu_harness


def _stack(d, heads, seq, d_in=72, d_out=136):
    return [wl.Layer(d_in, d), wl.norm_layer(d), wl.Layer(d, 3 * d), wl.attention_layer(d, heads, seq),
            wl.Layer(d, d, residual_src=1), wl.Layer(d, d_out)]


def _mask_all(layers):
    m = np.ones(2 * len(layers), dtype=np.uint8)
    for l, ly in enumerate(layers):
        if ly.kind == wl.KIND_ATTENTION:
            m[2 * l] = m[2 * l + 1] = 0
    return m


@pytest.mark.parametrize("heads,seq,batch", [(4, 50, 3), (2, 197, 2), (1, 208, 1), (2, 16, 5), (3, 1, 40), (2, 65, 3), (1, 256, 2), (2, 129, 2), (1, 128, 3)])
def test_all_trainable_tensors_selected(heads, seq, batch):
    # sequence lengths below, at and across the 128-row halves of a tile and the 16-column steps
    h = _h()
    layers = _stack(64 * heads, heads, seq)
    w = wl.small_stack(layers, batch * seq, wl.DT_BF16, 81, mask=_mask_all(layers), w_std=0.1, bias_std=0.05)
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)


@pytest.mark.parametrize("sel", [[10], [8, 9], [4, 5], [2, 3, 11], [0]])
def test_masks_around_the_attention_layer(sel):
    # deepest selected tensor above the attention layer (its backward does not run), directly above,
    # directly below (the QKV layer, whose dZ the attention backward writes), further down
    h = _h()
    layers = _stack(128, 2, 40)
    mask = np.zeros(12, dtype=np.uint8)
    mask[sel] = 1
    w = wl.small_stack(layers, 4 * 40, wl.DT_BF16, 82, mask=mask, w_std=0.1, bias_std=0.05)
    rep = h.check_step(w, mask, TOL_BF16, derived_w_tol=True)
    assert bool(rep.dgrad[3]) == (min(sel) // 2 < 3)


def test_full_vit_blocks_bf16():
    h = _h()
    w = wl.vit_b_full(seed=83, p_select=0.4, n_blocks=2, batch=3, seq=197, d=256, ffn=512, heads=4)
    if not w.mask.any():
        w.mask[-2:] = 1
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)
    m = _mask_all(w.layers)
    h.check_step(w, m, TOL_BF16, derived_w_tol=True)


def test_unsupported_shapes_and_selections_are_refused():
    ok = _stack(128, 2, 40)
    with pytest.raises(et.EtError):                                   # fp32 storage
        et.et_stack_create(ok, 80, wl.DT_F32)
    with pytest.raises(et.EtError):                                   # rows are not whole sequences
        et.et_stack_create(ok, 90, wl.DT_BF16)
    with pytest.raises(et.EtError):                                   # sequence too long
        et.et_stack_create(_stack(128, 2, 272), 544, wl.DT_BF16)
    with pytest.raises(et.EtError):                                   # head width is not 64
        et.et_stack_create([wl.Layer(64, 96), wl.Layer(96, 3 * 96), wl.attention_layer(96, 2, 8), wl.Layer(96, 8)], 16, wl.DT_BF16)
    with pytest.raises(et.EtError):                                   # last layer
        et.et_stack_create([wl.Layer(64, 384), wl.attention_layer(128, 2, 8)], 16, wl.DT_BF16)
    # a selection bit on the layer without tensors
    h = _h()
    w = wl.small_stack(ok, 80, wl.DT_BF16, 84, mask=_mask_all(ok), w_std=0.1)
    run = h.GpuRun(w)
    run.forward_loss()
    bad = w.mask.copy(); bad[6] = 1
    with pytest.raises(et.EtError):
        et.et_backward_elastic(run.stack, run.dY, bad, None, None, None, 0, 0.0, None)


def test_profiled_costs_follow_the_papers_rules_for_non_dense_layers():
    # Section 5.2: a normalisation layer's whole backward time sits in t_dy of beta; Section 5.3: the
    # attention core's backward time joins t_dy of the bias of the trainable layer below it
    import torch
    h = _h()
    layers = _stack(128, 2, 40)
    w = wl.small_stack(layers, 8 * 40, wl.DT_BF16, 85, mask=_mask_all(layers), w_std=0.1)
    run = h.GpuRun(w)
    run.forward_loss()
    t_dw, t_dy, t_fwd = et.et_profile_costs(run.stack, run.x, run.y, run.dY, iters=3)
    assert t_fwd > 0
    assert t_dw[2] == 0 and t_dw[3] == 0 and t_dy[2] == 0 and t_dy[3] > 0            # layer 1: normalisation
    assert t_dw[6] == 0 and t_dw[7] == 0 and t_dy[6] == 0 and t_dy[7] == 0            # layer 3: attention core
    assert t_dy[5] > 0                                                                # bias of the QKV layer below it
    for l in (0, 2, 4, 5):                                                            # dense layers
        assert t_dw[2 * l] > 0 and t_dw[2 * l + 1] > 0
        assert (t_dy[2 * l] > 0) == (l > 0)
    for l in (0, 4, 5):
        assert t_dy[2 * l + 1] == 0                                                   # a plain bias passes nothing on
    # the selector accepts these vectors as they are
    imp = np.abs(np.random.default_rng(0).normal(size=12))
    imp[6:8] = 0.0
    mask, val, est = et.et_select_dp(imp, t_dw, t_dy, t_fwd, 0.6, 1000)
    assert mask[6] == 0 and mask[7] == 0 and est <= 0.6 * (t_fwd + t_dw.sum() + t_dy.sum()) - t_fwd + 12 * (t_dw.sum() + t_dy.sum()) / 1000


def test_full_block_is_deterministic():
    # normalisation, attention and dense kernels: two runs from the same inputs give identical bits
    import torch
    h = _h()
    w = wl.vit_b_full(seed=86, p_select=0.5, n_blocks=2, batch=3, seq=197, d=128, ffn=256, heads=2)
    m = _mask_all(w.layers)
    outs = []
    for _ in range(2):
        run = h.GpuRun(w)
        run.forward_loss()
        grads = run.alloc_grads(m)
        delta = [h.to_dev(d, w.dtype) for d in wl.draw_delta(w, 4)]
        run.backward(m, grads, delta)
        outs.append(([g.clone() for g in grads if g is not None], run.importance.clone(), run.y.clone()))
    for a, b in zip(outs[0][0], outs[1][0]):
        assert torch.equal(a, b)
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])
