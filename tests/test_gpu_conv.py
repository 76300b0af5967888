"""Parity of k x k convolutions (patch-gather layer + dense layer) against the float64 oracle,
through the C ABI, on fp32 and bf16 stacks."""
import numpy as np
import pytest

import paper_2312_14227_b200 as et
import workloads as wl

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 2e-2


def _h():
    import gpu_harness
    return gpu_harness


def _mask_all(layers):
    m = np.ones(2 * len(layers), dtype=np.uint8)
    for l, ly in enumerate(layers):
        if ly.kind in (wl.KIND_IM2COL, wl.KIND_ATTENTION):
            m[2 * l] = m[2 * l + 1] = 0
    return m


def _conv_stack(act_mid, H=7, W=6):
    # gather as the first layer, after an activation layer, with its input feeding a residual, 5 x 5 and 1 x 1 taps
    return (wl.conv_layers(8, 64, H, W, 3, act=act_mid)                       # 0, 1
            + wl.conv_layers(64, 64, H, W, 3, act=wl.ACT_GELU_TANH)           # 2, 3: below it a layer with activation
            + [wl.Layer(64, 64, residual_src=2)]                              # 4: residual from the gather's input
            + wl.conv_layers(64, 72, H, W, 5)                                 # 5, 6
            + wl.conv_layers(72, 40, H, W, 1))                                # 7, 8


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, TOL_F32), (wl.DT_BF16, TOL_BF16)])
def test_all_trainable_tensors_selected(dtype, tol):
    h = _h()
    layers = _conv_stack(wl.ACT_RELU if dtype == wl.DT_F32 else wl.ACT_GELU_TANH)
    w = wl.small_stack(layers, 5 * 42, dtype, 91, mask=_mask_all(layers), w_std=0.06, bias_std=0.05)
    h.check_step(w, w.mask, tol, derived_w_tol=dtype == wl.DT_BF16)


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, TOL_F32), (wl.DT_BF16, TOL_BF16)])
@pytest.mark.parametrize("sel", [[16], [12, 13], [6, 7], [2], [3, 8], [2, 17]])
def test_masks_around_the_gather_layers(dtype, tol, sel):
    h = _h()
    layers = _conv_stack(wl.ACT_GELU_TANH)
    mask = np.zeros(2 * len(layers), dtype=np.uint8)
    mask[sel] = 1
    w = wl.small_stack(layers, 3 * 42, dtype, 92, mask=mask, w_std=0.06, bias_std=0.05)
    h.check_step(w, mask, tol, derived_w_tol=dtype == wl.DT_BF16)


def test_resnet_bottleneck_blocks_bf16():
    h = _h()
    w = wl.resnet_bottleneck(seed=93, p_select=0.5, n_blocks=2, images=4, height=14, width=14, c=256, mid=64)
    if not w.mask.any():
        w.mask[-2:] = 1
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)


def _folded_stack(H=7, W=6):
    """Gathers with 128 channels in front of a dense layer: on bf16 stacks the gathered matrix is never formed
    (the layer's three GEMMs fetch the patches by TMA in im2col mode).  Below the first one a layer with an
    activation, its input also feeding a residual; 3 x 3 and 5 x 5 taps; the last gather (64 channels) is formed."""
    return ([wl.Layer(24, 128, act=wl.ACT_GELU_TANH)]                          # 0
            + wl.conv_layers(128, 128, H, W, 3, act=wl.ACT_GELU_TANH)          # 1, 2
            + [wl.Layer(128, 128, residual_src=1)]                             # 3: residual from the gather's input
            + wl.conv_layers(128, 64, H, W, 5)                                 # 4, 5
            + wl.conv_layers(64, 40, H, W, 3))                                 # 6, 7


@pytest.mark.parametrize("images,H,W", [(10, 7, 6), (3, 14, 14), (1, 5, 9)])
def test_gathers_folded_into_the_gemms_bf16(images, H, W):
    # 128-row tiles start and end inside images; the last tile is ragged
    h = _h()
    layers = _folded_stack(H, W)
    w = wl.small_stack(layers, images * H * W, wl.DT_BF16, 94, mask=_mask_all(layers), w_std=0.06, bias_std=0.05)
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)


@pytest.mark.parametrize("sel", [[14], [10, 11], [4, 5], [6], [0], [1, 11]])
def test_masks_around_folded_gathers_bf16(sel):
    h = _h()
    layers = _folded_stack()
    mask = np.zeros(2 * len(layers), dtype=np.uint8)
    mask[sel] = 1
    w = wl.small_stack(layers, 6 * 42, wl.DT_BF16, 95, mask=mask, w_std=0.06, bias_std=0.05)
    h.check_step(w, mask, TOL_BF16, derived_w_tol=True)


def test_resnet_bottleneck_blocks_folded_gathers_bf16():
    h = _h()
    w = wl.resnet_bottleneck(seed=96, p_select=0.5, n_blocks=2, images=3, height=14, width=14, c=256, mid=128)
    if not w.mask.any():
        w.mask[-2:] = 1
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)


def test_unsupported_gathers_are_refused():
    with pytest.raises(et.EtError):                                   # even kernel size
        et.et_stack_create([wl.Layer(8, 32, kind=wl.KIND_IM2COL, height=4, width=4, ksize=2), wl.Layer(32, 8)], 16, wl.DT_F32)
    with pytest.raises(et.EtError):                                   # rows are not whole images
        et.et_stack_create(wl.conv_layers(8, 8, 4, 4, 3), 24, wl.DT_F32)
    with pytest.raises(et.EtError):                                   # channels not a multiple of 8
        et.et_stack_create(wl.conv_layers(12, 8, 4, 4, 3), 16, wl.DT_F32)
    with pytest.raises(et.EtError):                                   # nothing consumes the gathered rows
        et.et_stack_create([wl.Layer(8, 8), wl.Layer(8, 72, kind=wl.KIND_IM2COL, height=4, width=4, ksize=3)], 16, wl.DT_F32)
