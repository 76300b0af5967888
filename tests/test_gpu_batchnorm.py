"""Parity of batch normalisation layers (training mode; gamma and beta selectable tensors, Section 5.2)
against the float64 oracle, through the C ABI."""
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


def _bn_stack(dtype, d=72, hid=136):
    # batch norm with and without its activation, first in the stack, under a residual, before a fold, last
    act = wl.ACT_RELU if dtype == wl.DT_F32 else wl.ACT_GELU_TANH      # smooth on bf16 stacks (storage-rounding flips)
    return [
        wl.batchnorm_layer(d),
        wl.Layer(d, hid),
        wl.batchnorm_layer(hid, act),
        wl.Layer(hid, d, residual_src=0),
        wl.batchnorm_layer(d, eps=1e-3),
        wl.Layer(d, 3 * 256, fold=3),
        wl.Layer(256, d, act=wl.ACT_GELU_TANH, residual_src=4),
        wl.batchnorm_layer(d, wl.ACT_GELU_TANH),
    ]


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, TOL_F32), (wl.DT_BF16, TOL_BF16)])
def test_all_tensors_selected(dtype, tol):
    h = _h()
    w = wl.small_stack(_bn_stack(dtype), 333, dtype, 95, mask=np.ones(16, dtype=np.uint8), w_std=0.1, bias_std=0.05)
    h.check_step(w, w.mask, tol, derived_w_tol=dtype == wl.DT_BF16)


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, TOL_F32), (wl.DT_BF16, TOL_BF16)])
@pytest.mark.parametrize("sel", [[4], [5], [4, 5, 12], [0, 15], [1, 14], [15], [8, 9], [6]])
def test_masks_around_batchnorm_layers(dtype, tol, sel):
    h = _h()
    mask = np.zeros(16, dtype=np.uint8)
    mask[sel] = 1
    w = wl.small_stack(_bn_stack(dtype), 200, dtype, 96, mask=mask, w_std=0.1, bias_std=0.05)
    h.check_step(w, mask, tol, derived_w_tol=dtype == wl.DT_BF16)


@pytest.mark.parametrize("d,rows", [(8, 5), (264, 129), (1024, 300)])
def test_widths_and_row_counts(d, rows):
    h = _h()
    layers = [wl.Layer(64, d), wl.batchnorm_layer(d, wl.ACT_GELU_TANH), wl.Layer(d, 64), wl.batchnorm_layer(64)]
    for dtype, tol in ((wl.DT_BF16, TOL_BF16), (wl.DT_F32, TOL_F32)):
        w = wl.small_stack(layers, rows, dtype, 97, mask=np.ones(8, dtype=np.uint8), w_std=0.1, bias_std=0.05)
        h.check_step(w, w.mask, tol, derived_w_tol=dtype == wl.DT_BF16)


@pytest.mark.parametrize("dtype,tol,act", [(wl.DT_F32, TOL_F32, wl.ACT_RELU), (wl.DT_BF16, TOL_BF16, wl.ACT_GELU_TANH)])
def test_resnet_bottleneck_with_batchnorm(dtype, tol, act):
    # conv - batch norm - activation bottlenecks; ReLU on the fp32 stack, the smooth activation on the bf16 one
    # (a normalised pre-activation rounded to bf16 flips the ReLU derivative of about 1 % of the elements)
    h = _h()
    w = wl.resnet_bottleneck(seed=98, p_select=0.5, n_blocks=2, images=4, height=14, width=14, c=256, mid=64, bn=True,
                             act=act, dtype=dtype)
    if not w.mask.any():
        w.mask[-2:] = 1
    h.check_step(w, w.mask, tol, derived_w_tol=True)
