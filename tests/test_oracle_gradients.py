"""Pins of the oracle's floating-point parts against what mathematics fixes:
central finite differences of the loss, hand-computed 2x2 case, masked-vs-full
invariants, closed form of the importance sum, first-order Taylor identity."""
import numpy as np
import pytest

import workloads as wl
from oracle import elastic_oracle as orc


def _loss(layers, W, b, x, target):
    return orc.mse_loss(orc.forward(layers, W, b, x).a[-1], target)


def _all_kinds_stack():
    # every activation, a 3-way fold, two kinds of residual wiring, ragged widths
    return [
        wl.Layer(6, 9, fold=3),                                  # 0: fold, out width 3
        wl.Layer(3, 6, residual_src=0),                          # 1: residual from the stack input (width 6)
        wl.Layer(6, 10, act=wl.ACT_GELU_TANH),                   # 2
        wl.Layer(10, 6, residual_src=2),                         # 3: residual from a_2
        wl.Layer(6, 5, act=wl.ACT_RELU),                         # 4
        wl.Layer(5, 6, act=wl.ACT_GELU_TANH, residual_src=4),    # 5: activation AND residual
        wl.Layer(6, 4),                                          # 6
    ]


def _fd_check(layers, M, seed, h=1e-6, tol=2e-6):
    w = wl.small_stack(layers, M, wl.DT_F32, seed, w_std=0.4, bias_std=0.3)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    grads = orc.backward_full(w.layers, w.W, saved, dY)
    rng = np.random.default_rng(seed + 100)
    for l in range(len(layers)):
        for t, arr_list in ((2 * l, w.W), (2 * l + 1, w.b)):
            p = arr_list[l]
            g = grads[t]
            assert g.shape == p.shape
            if p.size == 0:                          # a layer without trainable tensors
                continue
            idxs = [tuple(rng.integers(0, s) for s in p.shape) for _ in range(12)]
            for idx in idxs:
                old = p[idx]
                p[idx] = old + h
                lp = _loss(w.layers, w.W, w.b, w.x, w.target)
                p[idx] = old - h
                lm = _loss(w.layers, w.W, w.b, w.x, w.target)
                p[idx] = old
                fd = (lp - lm) / (2 * h)
                if np.abs(g).max() < 1e-12:          # a gradient that is identically zero (a bias right before a
                    assert abs(fd) < 1e-7           # normalisation over the same axis): the difference quotient is noise
                    continue
                scale = max(abs(fd), np.abs(g).max() * 1e-3, 1e-12)
                assert abs(fd - g[idx]) / scale < tol, (l, t, idx, fd, g[idx])


def test_finite_differences_all_layer_kinds():
    _fd_check(_all_kinds_stack(), M=7, seed=11)


def test_finite_differences_vit_and_mlp_wiring():
    _fd_check(wl.vit_blocks(2, 6, 10), M=5, seed=5)
    _fd_check(wl.mlp_blocks(2, 4, 7, wl.ACT_RELU), M=6, seed=6)


def test_single_layer_by_hand():
    # L = 1, no activation: dW = X^T dY, db = column sums, checked entry by entry
    layers = [wl.Layer(2, 2)]
    X = np.array([[1.0, 2.0], [3.0, -1.0]])
    W = [np.array([[0.5, -1.0], [2.0, 0.25]])]
    b = [np.array([0.1, -0.2])]
    saved = orc.forward(layers, W, b, X)
    assert np.allclose(saved.a[1], [[1 * .5 + 2 * 2 + .1, -1 + .5 - .2], [1.5 - 2 + .1, -3 - .25 - .2]])
    dY = np.array([[1.0, 0.0], [0.0, 2.0]])
    g = orc.backward_full(layers, W, saved, dY)
    assert np.array_equal(g[0], [[1.0, 6.0], [2.0, -2.0]])
    assert np.array_equal(g[1], [1.0, 2.0])


def test_dgrad_orientation_two_layers_by_hand():
    # two linear layers: dW_0 = X^T (dY W_1^T); a transposed operand fails this
    layers = [wl.Layer(2, 3), wl.Layer(3, 2)]
    rng = np.random.default_rng(0)
    X, W0, W1 = rng.normal(size=(4, 2)), rng.normal(size=(2, 3)), rng.normal(size=(3, 2))
    dY = rng.normal(size=(4, 2))
    saved = orc.forward(layers, [W0, W1], [np.zeros(3), np.zeros(2)], X)
    g = orc.backward_full(layers, [W0, W1], saved, dY)
    want = np.zeros((2, 3))
    for i in range(2):
        for j in range(3):
            for m in range(4):
                for n in range(2):
                    want[i, j] += X[m, i] * dY[m, n] * W1[j, n]
    assert np.allclose(g[0], want, rtol=1e-12, atol=1e-12)


def test_gelu_tanh_known_values():
    # tanh-GELU at 0 is 0 with slope 1/2; for large |z| it tends to z and 0
    z = np.array([0.0, 10.0, -10.0, 1.0])
    v = orc.act_forward(z, orc.ACT_GELU_TANH)
    assert v[0] == 0.0 and abs(v[1] - 10.0) < 1e-12 and abs(v[2]) < 1e-12
    assert abs(v[3] - 0.8411919906082768) < 1e-12   # 0.5*(1+tanh(sqrt(2/pi)*1.044715))
    d = orc.act_derivative(z, orc.ACT_GELU_TANH)
    assert d[0] == 0.5 and abs(d[1] - 1.0) < 1e-9 and abs(d[2]) < 1e-9


def test_masked_is_subset_of_full_and_all_selected_is_full():
    w = wl.small_stack(_all_kinds_stack(), 9, wl.DT_F32, 3, w_std=0.3, bias_std=0.2)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    full = orc.backward_full(w.layers, w.W, saved, dY)
    rng = np.random.default_rng(0)
    for _ in range(20):
        mask = (rng.random(2 * w.L) < 0.3).astype(np.uint8)
        grads, plan = orc.backward_masked(w.layers, w.W, saved, dY, mask)
        assert sorted(grads) == [k for k in range(2 * w.L) if mask[k]]
        for k in grads:
            assert np.array_equal(grads[k], full[k])      # same arithmetic, bit-identical
    ones = np.ones(2 * w.L, dtype=np.uint8)
    grads, plan = orc.backward_masked(w.layers, w.W, saved, dY, ones)
    assert plan.deepest == 0 and plan.dgrad.sum() == w.L - 1
    for k in range(2 * w.L):
        assert np.array_equal(grads[k], full[k])


def test_importance_closed_form_for_gradient_step():
    # Eq. (2) with delta = -lr * g  =>  S_k = -lr * ||g_k||^2
    w = wl.small_stack(wl.vit_blocks(1, 6, 8), 5, wl.DT_F32, 8, w_std=0.3)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    full = orc.backward_full(w.layers, w.W, saved, dY)
    lr = 0.05
    delta = [-lr * full[k] for k in range(2 * w.L)]
    mask = np.ones(2 * w.L, dtype=np.uint8)
    S = orc.importance(full, delta, mask)
    for k in range(2 * w.L):
        assert abs(S[k] + lr * np.sum(full[k] ** 2)) <= 1e-14 * max(1.0, abs(S[k]))
    # independent delta: brute-force double loop on one kernel
    rng = np.random.default_rng(1)
    dl = [rng.normal(size=full[k].shape) for k in range(2 * w.L)]
    S = orc.importance(full, dl, mask)
    acc = 0.0
    for i in range(full[4].shape[0]):
        for j in range(full[4].shape[1]):
            acc += full[4][i, j] * dl[4][i, j]
    assert abs(acc - S[4]) < 1e-12
    # unselected tensors report 0
    mask[3] = 0
    assert orc.importance(full, dl, mask)[3] == 0.0


def test_importance_is_first_order_loss_change():
    # Eq. (6): L(w + dw) - L(w) = sum_k S_k + O(|dw|^2); the residual falls 4x when dw halves
    w = wl.small_stack(wl.mlp_blocks(2, 5, 9, wl.ACT_GELU_TANH), 6, wl.DT_F32, 4, w_std=0.4, bias_std=0.1)
    params = orc.tensors_of(w.W, w.b)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    L0, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    full = orc.backward_full(w.layers, w.W, saved, dY)
    mask = np.ones(2 * w.L, dtype=np.uint8)
    res = []
    for lr in (0.004, 0.002, 0.001):
        delta = [-lr * full[k] for k in range(2 * w.L)]
        S = orc.importance(full, delta, mask).sum()
        new = orc.sgd_masked(params, full, mask, lr)
        L1 = _loss(w.layers, new[0::2], new[1::2], w.x, w.target)
        assert L1 < L0 and S < 0
        res.append((L1 - L0) - S)
    assert 3.5 < res[0] / res[1] < 4.5 and 3.5 < res[1] / res[2] < 4.5
    assert abs(res[2]) < 0.05 * abs(S)


def test_sgd_masked_leaves_frozen_tensors_alone():
    w = wl.small_stack(wl.mlp_blocks(1, 4, 6, wl.ACT_RELU), 3, wl.DT_F32, 2)
    params = orc.tensors_of(w.W, w.b)
    grads = {k: np.ones_like(p) for k, p in enumerate(params)}
    mask = np.array([1, 0, 0, 1], dtype=np.uint8)
    new = orc.sgd_masked(params, grads, mask, 0.5)
    assert new[1] is params[1] and new[2] is params[2]
    assert np.array_equal(new[0], params[0] - 0.5) and np.array_equal(new[3], params[3] - 0.5)


def test_mse_gradient_normalisation():
    y = np.array([[1.0, 2.0], [3.0, 5.0]])
    t = np.zeros((2, 2))
    loss, g = orc.mse_loss_grad(y, t)
    assert loss == (1 + 4 + 9 + 25) / 4 and np.array_equal(g, y / 2)


# ------------------------------------------------------------------ normalisation layers (Section 5.2)
def _norm_stack():
    # normalisation first, between dense layers, before an activation layer, under a residual, last
    return [
        wl.norm_layer(6),                                        # 0: acts on the stack input
        wl.Layer(6, 8, act=wl.ACT_GELU_TANH),                    # 1
        wl.Layer(8, 6, residual_src=0),                          # 2: residual from the stack input
        wl.norm_layer(6, eps=1e-3),                              # 3: its input a_3 also feeds layer 5's residual
        wl.Layer(6, 9, fold=3),                                  # 4
        wl.Layer(3, 6, act=wl.ACT_RELU, residual_src=3),         # 5
        wl.norm_layer(6),                                        # 6: last layer
    ]


def test_finite_differences_through_normalisation_layers():
    _fd_check(_norm_stack(), M=5, seed=21, tol=5e-6)
    _fd_check(wl.vit_blocks_prenorm(2, 6, 10), M=4, seed=22, tol=5e-6)


def test_normalisation_forward_closed_forms():
    # two features: xhat = +-(|a-b|/2) / sqrt((a-b)^2/4 + eps), whatever the row's mean
    ly = [wl.norm_layer(2, eps=0.25)]
    x = np.array([[3.0, 1.0], [-2.0, 6.0], [5.0, 5.0]])
    gamma, beta = np.array([2.0, -1.0]), np.array([0.5, 0.25])
    y = orc.forward(ly, [gamma], [beta], x).a[-1]
    half = np.array([1.0, 4.0, 0.0])
    xh = half / np.sqrt(half ** 2 + 0.25)
    want = np.stack([np.array([s, -s]) * gamma + beta for s in (xh[0], -xh[1], 0.0)])
    assert np.allclose(y, want, atol=1e-15)
    # any width: rows of xhat have mean 0 and second moment var/(var+eps); shifting or scaling a row
    # (eps = 0) does not change the output
    rng = np.random.default_rng(3)
    x = rng.normal(size=(9, 11)) * 3.0 + 2.0
    ly = [wl.norm_layer(11, eps=0.0)]
    one, zero = np.ones(11), np.zeros(11)
    xh = orc.forward(ly, [one], [zero], x).a[-1]
    assert np.allclose(xh.mean(axis=1), 0.0, atol=1e-14) and np.allclose((xh ** 2).mean(axis=1), 1.0, atol=1e-13)
    assert np.allclose(orc.forward(ly, [one], [zero], 7.5 * x - 4.0).a[-1], xh, atol=1e-12)


def test_normalisation_gradients_match_the_library_layer_norm():
    # the same stack written with torch's own linear / layer_norm / gelu and differentiated by autograd
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    layers = [wl.Layer(5, 8), wl.norm_layer(8, eps=1e-5), wl.Layer(8, 8, act=wl.ACT_GELU_TANH), wl.norm_layer(8, eps=1e-2)]
    w = wl.small_stack(layers, 6, wl.DT_F32, 31, w_std=0.5, bias_std=0.2)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    grads = orc.backward_full(w.layers, w.W, saved, dY)
    tW = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in w.W]
    tb = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in w.b]
    h = torch.tensor(w.x, dtype=torch.float64)
    for l, ly in enumerate(layers):
        if ly.kind == wl.KIND_NORM:
            h = F.layer_norm(h, (ly.out_features,), tW[l], tb[l], ly.eps)
        else:
            h = h @ tW[l] + tb[l]
            if ly.act == wl.ACT_GELU_TANH:
                h = F.gelu(h, approximate="tanh")
    loss = ((h - torch.tensor(w.target, dtype=torch.float64)) ** 2).mean()
    loss.backward()
    assert abs(loss.item() - orc.mse_loss(saved.a[-1], w.target)) < 1e-13
    for l in range(len(layers)):
        assert np.allclose(grads[2 * l], tW[l].grad.numpy(), rtol=1e-9, atol=1e-13), l
        assert np.allclose(grads[2 * l + 1], tb[l].grad.numpy(), rtol=1e-9, atol=1e-13), l


def test_masked_backward_with_normalisation_layers():
    # selected tensors get the full-backprop gradients; nothing below the deepest selected layer runs;
    # a normalisation layer that is itself the deepest passes no gradient on
    layers = _norm_stack()
    w = wl.small_stack(layers, 5, wl.DT_F32, 23, w_std=0.4, bias_std=0.3)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    full = orc.backward_full(w.layers, w.W, saved, dY)
    mask = np.zeros(14, dtype=np.uint8)
    mask[[6, 7, 10, 13]] = 1                     # gamma_3, beta_3, W_5, beta_6
    grads, plan = orc.backward_masked(w.layers, w.W, saved, dY, mask)
    assert plan.deepest == 3 and list(plan.dgrad) == [False] * 4 + [True] * 3
    assert sorted(grads) == [6, 7, 10, 13]
    for t in grads:
        assert np.array_equal(grads[t], full[t])
    assert orc.executed_flops(layers, 5, plan) == 2.0 * 5 * (6 * 9 + 2 * 3 * 6)


def test_magnitude_metric_is_the_l1_norm():
    tensors = [np.array([[1.0, -2.0], [0.5, 0.0]]), np.array([-3.0, 4.0]), np.array([7.0])]
    assert orc.magnitude_metric(tensors, [1, 1, 0]).tolist() == [3.5, 7.0, 0.0]
    # unlike Eq. 2 it is not additive over a split of the update, and it ignores the sign of the effect
    assert orc.magnitude_metric([-tensors[0]], [1])[0] == 3.5


# ------------------------------------------------------------------ attention core (non-trainable layer)
def _attn_stack(d=8, heads=2, seq=5):
    return [wl.Layer(6, d), wl.norm_layer(d), wl.Layer(d, 3 * d), wl.attention_layer(d, heads, seq),
            wl.Layer(d, d, residual_src=1), wl.Layer(d, 4)]


def test_finite_differences_through_the_attention_core():
    _fd_check(_attn_stack(), M=15, seed=41, tol=5e-6)
    _fd_check(wl.vit_blocks_full(1, 8, 12, heads=2, seq=4), M=12, seed=42, tol=5e-6)


def test_attention_matches_the_library_scaled_dot_product_attention():
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    d, H, S, B = 12, 3, 7, 4
    layers = [wl.Layer(5, 3 * d), wl.attention_layer(d, H, S), wl.Layer(d, 6)]
    w = wl.small_stack(layers, B * S, wl.DT_F32, 43, w_std=0.6, bias_std=0.2)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    grads = orc.backward_full(w.layers, w.W, saved, dY)
    tW = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (w.W[0], w.W[2])]
    tb = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (w.b[0], w.b[2])]
    qkv = torch.tensor(w.x, dtype=torch.float64) @ tW[0] + tb[0]
    q, k, v = (qkv[:, i * d:(i + 1) * d].reshape(B, S, H, d // H).transpose(1, 2) for i in range(3))
    o = F.scaled_dot_product_attention(q, k, v).transpose(1, 2).reshape(B * S, d)
    assert np.allclose(o.detach().numpy(), saved.a[2], rtol=1e-10, atol=1e-12)
    loss = ((o @ tW[1] + tb[1] - torch.tensor(w.target, dtype=torch.float64)) ** 2).mean()
    loss.backward()
    for t, ref in ((0, tW[0]), (1, tb[0]), (4, tW[1]), (5, tb[1])):
        assert np.allclose(grads[t], ref.grad.numpy(), rtol=1e-9, atol=1e-13), t
    assert grads[2].size == 0 and grads[3].size == 0


def test_attention_closed_forms():
    # equal keys: the softmax is uniform and every query gets the mean of the values; one key far ahead:
    # the output is that key's value; sequences do not mix
    d, H, S = 4, 1, 3
    ly = [wl.attention_layer(d, H, S)]
    q = np.arange(24.0).reshape(6, 4) / 10
    k = np.ones((6, 4))
    v = np.array([[1.0, 0, 0, 0], [0, 1, 0, 0], [0, 0, 1, 0], [5, 5, 5, 5], [7, 7, 7, 7], [9, 9, 9, 9]])
    o = orc.forward(ly, [np.zeros(0)], [np.zeros(0)], np.concatenate([q, k, v], axis=1)).a[-1]
    assert np.allclose(o[:3], np.tile(v[:3].mean(0), (3, 1))) and np.allclose(o[3:], np.tile(v[3:].mean(0), (3, 1)))
    k2 = k.copy(); k2[1] = 1000.0
    q2 = np.ones((6, 4))
    o = orc.forward(ly, [np.zeros(0)], [np.zeros(0)], np.concatenate([q2, k2, v], axis=1)).a[-1]
    assert np.allclose(o[:3], np.tile(v[1], (3, 1))) and np.allclose(o[3:], np.tile(v[3:].mean(0), (3, 1)))


# ------------------------------------------------------------------ k x k convolution = patch gather + dense layer
def test_convolution_matches_the_library_conv2d():
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    n, H, W, cin, cmid, cout, k = 2, 5, 4, 3, 6, 4, 3
    layers = [wl.Layer(cin, cmid, act=wl.ACT_RELU)] + wl.conv_layers(cmid, cout, H, W, k, act=wl.ACT_GELU_TANH) + \
        wl.conv_layers(cout, 5, H, W, 5)
    w = wl.small_stack(layers, n * H * W, wl.DT_F32, 61, w_std=0.5, bias_std=0.2)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    grads = orc.backward_full(w.layers, w.W, saved, dY)
    tW = {l: torch.tensor(w.W[l], dtype=torch.float64, requires_grad=True) for l in (0, 2, 4)}
    tb = {l: torch.tensor(w.b[l], dtype=torch.float64, requires_grad=True) for l in (0, 2, 4)}
    h = torch.relu(torch.tensor(w.x, dtype=torch.float64) @ tW[0] + tb[0])
    img = h.reshape(n, H, W, cmid).permute(0, 3, 1, 2)                            # NCHW for the library
    k1 = tW[2].reshape(k, k, cmid, cout).permute(3, 2, 0, 1)                       # (kh, kw, cin, cout) -> OIHW
    img = F.gelu(F.conv2d(img, k1, tb[2], padding=k // 2), approximate="tanh")
    k2 = tW[4].reshape(5, 5, cout, 5).permute(3, 2, 0, 1)
    img = F.conv2d(img, k2, tb[4], padding=2)
    y = img.permute(0, 2, 3, 1).reshape(n * H * W, 5)
    assert np.allclose(y.detach().numpy(), saved.a[-1], rtol=1e-10, atol=1e-12)
    loss = ((y - torch.tensor(w.target, dtype=torch.float64)) ** 2).mean()
    loss.backward()
    for l in (0, 2, 4):
        assert np.allclose(grads[2 * l], tW[l].grad.numpy(), rtol=1e-9, atol=1e-13), l
        assert np.allclose(grads[2 * l + 1], tb[l].grad.numpy(), rtol=1e-9, atol=1e-13), l


def test_finite_differences_through_convolutions():
    layers = [wl.Layer(3, 4, act=wl.ACT_GELU_TANH)] + wl.conv_layers(4, 4, 3, 4, 3, act=wl.ACT_RELU) + \
        [wl.Layer(4, 4, residual_src=1)] + wl.conv_layers(4, 2, 3, 4, 3)
    _fd_check(layers, M=2 * 12, seed=62, tol=5e-6)


def test_patch_gather_closed_forms():
    # a 1 x 1 "convolution" gathers nothing but the pixel itself; a 3 x 3 gather of a one-hot image puts the
    # hot pixel into tap (2 - dh, 2 - dw) of its neighbour at offset (dh - 1, dw - 1); borders see zeros
    x = np.arange(2 * 3 * 3 * 2, dtype=np.float64).reshape(18, 2)
    one = [wl.Layer(2, 2, kind=wl.KIND_IM2COL, height=3, width=3, ksize=1)]
    assert np.array_equal(orc.forward(one, [np.zeros(0)], [np.zeros(0)], x).a[-1], x)
    hot = np.zeros((9, 1)); hot[4] = 1.0                                           # centre of a 3 x 3 image
    g = [wl.Layer(1, 9, kind=wl.KIND_IM2COL, height=3, width=3, ksize=3)]
    col = orc.forward(g, [np.zeros(0)], [np.zeros(0)], hot).a[-1]
    assert np.array_equal(col, np.eye(9)[::-1])                                   # pixel p sees the centre in tap 8 - p
    corner = np.zeros((9, 1)); corner[0] = 1.0
    col = orc.forward(g, [np.zeros(0)], [np.zeros(0)], corner).a[-1]
    assert col.sum() == 4 and col[0, 4] == 1 and col[1, 3] == 1 and col[3, 1] == 1 and col[4, 0] == 1


# ------------------------------------------------------------------ batch normalisation (Section 5.2)
def test_batchnorm_matches_the_library_batch_norm():
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    layers = [wl.Layer(5, 8), wl.batchnorm_layer(8, wl.ACT_RELU, eps=1e-5), wl.Layer(8, 6, act=wl.ACT_GELU_TANH),
              wl.batchnorm_layer(6, eps=1e-2), wl.Layer(6, 4)]
    w = wl.small_stack(layers, 9, wl.DT_F32, 71, w_std=0.5, bias_std=0.2)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    grads = orc.backward_full(w.layers, w.W, saved, dY)
    tW = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in w.W]
    tb = [torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in w.b]
    h = torch.tensor(w.x, dtype=torch.float64)
    for l, ly in enumerate(layers):
        if ly.kind == wl.KIND_BATCHNORM:
            h = F.batch_norm(h, None, None, tW[l], tb[l], training=True, eps=ly.eps)
        else:
            h = h @ tW[l] + tb[l]
        if ly.act == wl.ACT_RELU:
            h = torch.relu(h)
        elif ly.act == wl.ACT_GELU_TANH:
            h = F.gelu(h, approximate="tanh")
    loss = ((h - torch.tensor(w.target, dtype=torch.float64)) ** 2).mean()
    loss.backward()
    assert abs(loss.item() - orc.mse_loss(saved.a[-1], w.target)) < 1e-13
    for l in range(len(layers)):
        assert np.allclose(grads[2 * l], tW[l].grad.numpy(), rtol=1e-8, atol=1e-13), l
        assert np.allclose(grads[2 * l + 1], tb[l].grad.numpy(), rtol=1e-8, atol=1e-13), l


def test_finite_differences_through_batchnorm():
    layers = [wl.Layer(4, 6), wl.batchnorm_layer(6, wl.ACT_GELU_TANH), wl.Layer(6, 6, residual_src=2),
              wl.batchnorm_layer(6, eps=1e-3), wl.Layer(6, 3)]
    _fd_check(layers, M=7, seed=72, tol=5e-6)
    _fd_check(wl.resnet_bottleneck_blocks(1, 8, 4, 3, 3, bn=True), M=18, seed=73, tol=5e-6)


def test_batchnorm_closed_forms():
    # every column of xhat has mean 0 and second moment var / (var + eps) over the rows; a per-column shift
    # and scale of the input (eps = 0) leaves the output unchanged; two rows give xhat = +-1
    rng = np.random.default_rng(5)
    x = rng.normal(size=(11, 4)) * 3.0 + 2.0
    ly = [wl.batchnorm_layer(4, eps=0.0)]
    one, zero = np.ones(4), np.zeros(4)
    xh = orc.forward(ly, [one], [zero], x).a[-1]
    assert np.allclose(xh.mean(axis=0), 0.0, atol=1e-14) and np.allclose((xh ** 2).mean(axis=0), 1.0, atol=1e-13)
    assert np.allclose(orc.forward(ly, [one], [zero], x * np.array([2.0, 0.5, 7.0, 1.0]) + 3.0).a[-1], xh, atol=1e-12)
    two = orc.forward(ly, [np.array([2.0, 3.0, 4.0, 5.0])], [np.array([1.0, 1.0, 1.0, 1.0])], np.array([[1.0, 5, 2, 0], [3.0, 1, 8, 4]])).a[-1]
    assert np.allclose(two, [[-1.0, 4.0, -3.0, -4.0], [3.0, -2.0, 5.0, 6.0]])
