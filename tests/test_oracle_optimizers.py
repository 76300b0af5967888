"""Pins of the oracle's masked optimisers against closed forms of the published algorithms."""
import numpy as np

from oracle import elastic_oracle as orc


def _setup(seed=0):
    rng = np.random.default_rng(seed)
    params = [rng.normal(size=(3, 4)), rng.normal(size=4), rng.normal(size=(2, 2))]
    grads = {k: rng.normal(size=p.shape) for k, p in enumerate(params)}
    return params, grads


def test_sgdw_reduces_to_sgd_and_to_pure_decay():
    params, grads = _setup()
    mask = [1, 1, 1]
    st = orc.optimizer_state(params)
    new = orc.optimizer_step_masked(params, grads, mask, orc.OPT_SGDW, 0.1, st, momentum=0.0, wd=0.0)
    ref = orc.sgd_masked(params, grads, mask, 0.1)
    for a, b in zip(new, ref):
        assert np.allclose(a, b, rtol=1e-15, atol=0)
    # zero gradient: the weights shrink geometrically, (1 - wd)^t
    zero = {k: np.zeros_like(p) for k, p in enumerate(params)}
    st = orc.optimizer_state(params)
    cur = params
    for t in range(5):
        cur = orc.optimizer_step_masked(cur, zero, mask, orc.OPT_SGDW, 0.1, st, momentum=0.9, wd=0.01)
    for a, p in zip(cur, params):
        assert np.allclose(a, p * 0.99 ** 5, rtol=1e-14)


def test_sgdw_momentum_is_a_geometric_series_for_a_constant_gradient():
    params, grads = _setup(1)
    mask = [1, 1, 1]
    st = orc.optimizer_state(params)
    cur, lr, mu, T = params, 0.05, 0.9, 6
    for t in range(T):
        cur = orc.optimizer_step_masked(cur, grads, mask, orc.OPT_SGDW, lr, st, momentum=mu, wd=0.0)
    # m_t = lr g (1 - mu^t)/(1 - mu);  w_T = w_0 - sum_t m_t
    total = sum(lr * (1 - mu ** t) / (1 - mu) for t in range(1, T + 1))
    for k, p in enumerate(params):
        assert np.allclose(cur[k], p - total * grads[k], rtol=1e-13)
        assert np.allclose(st[0][k], lr * grads[k] * (1 - mu ** T) / (1 - mu), rtol=1e-13)


def test_adam_constant_gradient_moves_by_lr_per_step():
    # with a constant gradient the bias-corrected moments are g and g^2 at every step:
    # w_T = w_0 - T * lr * g / (|g| + eps)
    params, grads = _setup(2)
    mask = [1, 1, 1]
    st = orc.optimizer_state(params)
    cur, lr, T, eps = params, 1e-3, 7, 1e-8
    for t in range(1, T + 1):
        cur = orc.optimizer_step_masked(cur, grads, mask, orc.OPT_ADAM, lr, st, step=t, eps=eps)
    for k, p in enumerate(params):
        assert np.allclose(cur[k], p - T * lr * grads[k] / (np.abs(grads[k]) + eps), rtol=1e-10, atol=1e-14)


def test_masked_update_leaves_unselected_tensors_and_state_alone():
    params, grads = _setup(3)
    for kind in (orc.OPT_SGD, orc.OPT_SGDW, orc.OPT_ADAM):
        st = orc.optimizer_state(params)
        new = orc.optimizer_step_masked(params, grads, [1, 0, 1], kind, 0.1, st, wd=0.01)
        assert new[1] is params[1]
        assert not st[0][1].any() and not st[1][1].any()
        assert not np.array_equal(new[0], params[0]) and not np.array_equal(new[2], params[2])
