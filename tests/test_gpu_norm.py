"""Parity of normalisation layers as stack members (gamma and beta are selectable tensors)
against the float64 oracle, through the C ABI.  Same bars as the dense-layer parity tests; gamma is near 1, where a bf16 store alone is off by up
to 2^-9, so bf16 stacks take the derived weight bound."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 2e-2


def _h():
    import gpu_harness
    return gpu_harness


def _norm_stack(dtype, d=72, hid=136):
    # normalisation first, before an activation layer, under a residual, between dense layers, last.
    # bf16 stacks take the smooth activation in layer 5: six layers of bf16 storage rounding move its
    # pre-activations by about 0.3 %, which flips the ReLU derivative (0 <-> 1) of about that share of
    # the elements and alone puts 5 % rms error into everything below (checked on the CPU by rounding
    # the oracle's intermediates to bf16)
    act5 = wl.ACT_RELU if dtype == wl.DT_F32 else wl.ACT_GELU_TANH
    return [
        wl.norm_layer(d),
        wl.Layer(d, hid, act=wl.ACT_GELU_TANH),
        wl.Layer(hid, d, residual_src=0),
        wl.norm_layer(d, eps=1e-3),
        wl.Layer(d, 3 * 256, fold=3),
        wl.Layer(256, d, act=act5, residual_src=3),
        wl.norm_layer(d),
    ]


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, TOL_F32), (wl.DT_BF16, TOL_BF16)])
def test_all_tensors_selected(dtype, tol):
    h = _h()
    w = wl.small_stack(_norm_stack(dtype), 333, dtype, 51, mask=np.ones(14, dtype=np.uint8), w_std=0.1, bias_std=0.05)
    h.check_step(w, w.mask, tol, derived_w_tol=dtype == wl.DT_BF16)


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, TOL_F32), (wl.DT_BF16, TOL_BF16)])
@pytest.mark.parametrize("sel", [[6], [7], [6, 7, 10], [0, 13], [1, 12], [13], [4, 5]])
def test_masks_around_normalisation_layers(dtype, tol, sel):
    # the deepest selected tensor is a gamma, a beta, a kernel below / above a normalisation layer ...
    h = _h()
    mask = np.zeros(14, dtype=np.uint8)
    mask[sel] = 1
    w = wl.small_stack(_norm_stack(dtype), 200, dtype, 52, mask=mask, w_std=0.1, bias_std=0.05)
    h.check_step(w, mask, tol, derived_w_tol=dtype == wl.DT_BF16)


@pytest.mark.parametrize("d", [8, 256, 264, 1024, 1536, 2048])
def test_feature_widths(d):
    # one to eight register chunks per lane, ragged last chunk
    h = _h()
    layers = [wl.Layer(64, d), wl.norm_layer(d), wl.Layer(d, 64), wl.norm_layer(64)]
    w = wl.small_stack(layers, 77, wl.DT_BF16, 53, mask=np.ones(8, dtype=np.uint8), w_std=0.1, bias_std=0.05)
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)
    w = wl.small_stack(layers, 77, wl.DT_F32, 54, mask=np.ones(8, dtype=np.uint8), w_std=0.1, bias_std=0.05)
    h.check_step(w, w.mask, TOL_F32)


def test_prenorm_vit_blocks_bf16():
    h = _h()
    w = wl.vit_b_prenorm(seed=61, p_select=0.4, n_blocks=2, tokens=700, d=256, ffn=512)
    if not w.mask.any():
        w.mask[-2:] = 1
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)
    w.mask[:] = 1
    h.check_step(w, w.mask, TOL_BF16, derived_w_tol=True)


def test_wider_than_supported_is_refused():
    import paper_2312_14227_b200 as et
    with pytest.raises(et.EtError):
        et.et_stack_create([wl.norm_layer(2056)], 16, wl.DT_BF16)
    with pytest.raises(et.EtError):
        et.et_stack_create([wl.Layer(8, 12, kind=wl.KIND_NORM)], 16, wl.DT_F32)
