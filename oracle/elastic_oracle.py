"""CPU oracle for the elastic (masked) backward pass of a stack of dense layers.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain float64 statement of what
the CUDA library computes.  It shares no code with the CUDA path and must never be
imported by it; only tests, the smoke check and the benchmark's CPU-baseline leg
use it.  numpy's matmul is the one library primitive used as a step.

Conventions (the paper, Sections 2.2, 3.3 and 5): layers and tensors are indexed
in forward execution order, 0 = nearest the input.  Tensor 2*l is the kernel of
layer l, tensor 2*l+1 its bias.  Layer l computes

    Z_l     = a_l @ W_l + b_l                       a_l : [M, K_l], W_l : [K_l, N_l]
    H_l     = act_l(Z_l)
    a_{l+1} = sum of `fold` equal column slices of H_l  (+ a_j if residual_src = j)

or, for a normalisation layer (Section 5.2; its Gamma and Beta are tensors 2*l and 2*l+1),

    xhat    = (a_l - mean) / sqrt(var + eps)         mean, var over the features of each row
    a_{l+1} = xhat * gamma_l + beta_l

or, for a batch normalisation layer (Section 5.2's subject; training mode, no running averages),

    xhat    = (a_l - mean) / sqrt(var + eps)         mean, biased var of each feature over all rows
    a_{l+1} = act_l( xhat * gamma_l + beta_l )

or, for a patch-gather layer (no trainable tensors; with the dense layer after it, it is a k x k
convolution with stride 1 and zero padding k // 2 on NHWC rows, the convolutional layer of Section 5.1),

    a_{l+1}[(n,h,w), (kh*k + kw)*C + c] = a_l[(n, h + kh - k//2, w + kw - k//2), c]     (0 outside the image)

or, for an attention layer (no trainable tensors; Sections 5.3 / 5.4 count attention operations as
non-trainable layers), with a_l = [q | k | v] (three blocks of `heads * head_dim` columns) and the
rows grouped into sequences of `seq` consecutive tokens,

    P       = softmax_over_keys( q_h k_h^T / sqrt(head_dim) )      per sequence and head h
    a_{l+1} = [ P v_h ]_h                                          heads side by side

Pins (tests/test_oracle_*.py): central finite differences of the loss for every
tensor and every layer kind; the closed form of the importance sum when the update
is a gradient step; the first-order Taylor identity of Eq. (6); masked == full
backprop on the selected tensors and all-selected == full; the two worked examples
the paper prints for the time model (Section 2.2) and for f(M) (Eq. 3); brute-force
enumeration for the selector.  The paper prints no numeric gradients or importances,
so beyond those pins the values are unpinned against the paper itself.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np

ACT_NONE, ACT_GELU_TANH, ACT_RELU = 0, 1, 2
KIND_DENSE, KIND_NORM, KIND_ATTENTION, KIND_IM2COL, KIND_BATCHNORM = 0, 1, 2, 3, 4
STRICT, INCLUSIVE = 0, 1


def _kind(ly) -> int:
    return getattr(ly, "kind", KIND_DENSE)

_C0 = np.sqrt(2.0 / np.pi)
_C1 = 0.044715


# --------------------------------------------------------------------------- activations
def act_forward(z: np.ndarray, act: int) -> np.ndarray:
    if act == ACT_NONE:
        return z
    if act == ACT_RELU:
        return np.where(z > 0.0, z, 0.0)
    if act == ACT_GELU_TANH:
        # tanh form of GELU: 0.5 z (1 + tanh( sqrt(2/pi) (z + 0.044715 z^3) ))
        return 0.5 * z * (1.0 + np.tanh(_C0 * (z + _C1 * z ** 3)))
    raise ValueError(act)


def act_derivative(z: np.ndarray, act: int) -> np.ndarray:
    if act == ACT_NONE:
        return np.ones_like(z)
    if act == ACT_RELU:
        return np.where(z > 0.0, 1.0, 0.0)
    if act == ACT_GELU_TANH:
        u = _C0 * (z + _C1 * z ** 3)
        t = np.tanh(u)
        du = _C0 * (1.0 + 3.0 * _C1 * z ** 2)
        return 0.5 * (1.0 + t) + 0.5 * z * (1.0 - t * t) * du
    raise ValueError(act)


# --------------------------------------------------------------------------- forward
@dataclass
class Saved:
    a: List[np.ndarray]    # a[0] = input, a[l+1] = output of layer l
    Z: List[np.ndarray]    # pre-activations


def forward(layers, W: Sequence[np.ndarray], b: Sequence[np.ndarray], x: np.ndarray) -> Saved:
    """Forward pass of every layer (the forward time is the same for any selection,
    Eq. 3), keeping what the backward pass needs."""
    a = [np.asarray(x, dtype=np.float64)]
    Z = []
    for l, ly in enumerate(layers):
        if _kind(ly) == KIND_BATCHNORM:
            # batch normalisation, training mode: mean and biased variance of each feature over all rows;
            # Z keeps (xhat, 1/sqrt(var + eps), pre-activation)
            mean = a[l].mean(axis=0, keepdims=True)
            var = ((a[l] - mean) ** 2).mean(axis=0, keepdims=True)
            rstd = 1.0 / np.sqrt(var + ly.eps)
            xhat = (a[l] - mean) * rstd
            z = xhat * np.asarray(W[l], dtype=np.float64) + np.asarray(b[l], dtype=np.float64)
            Z.append((xhat, rstd, z))
            a.append(act_forward(z, ly.act))
            continue
        if _kind(ly) == KIND_IM2COL:
            # patch gather of a k x k convolution, stride 1, zero padding k // 2, on NHWC rows:
            # col[(n,h,w), (kh*k + kw)*C + c] = x[n, h + kh - p, w + kw - p, c]  (0 outside the image)
            C_, Hh, Ww, k = ly.in_features, ly.height, ly.width, ly.ksize
            pd = k // 2
            xi = a[l].reshape(-1, Hh, Ww, C_)
            xp = np.zeros((xi.shape[0], Hh + 2 * pd, Ww + 2 * pd, C_))
            xp[:, pd:pd + Hh, pd:pd + Ww, :] = xi
            col = np.concatenate([xp[:, kh:kh + Hh, kw:kw + Ww, :] for kh in range(k) for kw in range(k)], axis=3)
            Z.append(None)
            a.append(col.reshape(a[l].shape[0], k * k * C_))
            continue
        if _kind(ly) == KIND_ATTENTION:
            d = ly.out_features
            H, S = ly.heads, ly.seq
            dh = d // H
            B = a[l].shape[0] // S
            q, k, v = (a[l][:, i * d:(i + 1) * d].reshape(B, S, H, dh).transpose(0, 2, 1, 3) for i in range(3))
            s_ = q @ k.transpose(0, 1, 3, 2) / np.sqrt(dh)                  # [B, H, S(query), S(key)]
            s_ = s_ - s_.max(axis=-1, keepdims=True)
            P = np.exp(s_)
            P = P / P.sum(axis=-1, keepdims=True)
            o = (P @ v).transpose(0, 2, 1, 3).reshape(B * S, d)
            Z.append((P, q, k, v))
            a.append(o)
            continue
        if _kind(ly) == KIND_NORM:
            # layer normalisation: per row, biased variance; Z keeps (xhat, 1/sqrt(var + eps))
            mean = a[l].mean(axis=1, keepdims=True)
            var = ((a[l] - mean) ** 2).mean(axis=1, keepdims=True)
            rstd = 1.0 / np.sqrt(var + ly.eps)
            xhat = (a[l] - mean) * rstd
            Z.append((xhat, rstd))
            a.append(xhat * np.asarray(W[l], dtype=np.float64) + np.asarray(b[l], dtype=np.float64))
            continue
        z = a[l] @ np.asarray(W[l], dtype=np.float64) + np.asarray(b[l], dtype=np.float64)
        h = act_forward(z, ly.act)
        w = ly.out_features // ly.fold
        out = np.zeros((h.shape[0], w))
        for s in range(ly.fold):
            out = out + h[:, s * w:(s + 1) * w]
        if ly.residual_src >= 0:
            out = out + a[ly.residual_src]
        Z.append(z)
        a.append(out)
    return Saved(a=a, Z=Z)


def mse_loss(y: np.ndarray, target: np.ndarray) -> float:
    """Mean over all M*D elements of (y - target)^2."""
    return float(np.mean((y - target) ** 2))


def mse_loss_grad(y: np.ndarray, target: np.ndarray):
    n = y.size
    return mse_loss(y, target), 2.0 * (y - target) / n


# --------------------------------------------------------------------------- which work runs
@dataclass
class Plan:
    deepest: int               # smallest layer index owning a selected tensor; L if none
    dgrad: np.ndarray          # bool[L]  error gradient passed through layer l (dX_l computed)
    wgrad: np.ndarray          # bool[L]  kernel gradient computed
    bgrad: np.ndarray          # bool[L]  bias gradient computed
    updated: np.ndarray        # bool[2L] tensor written by the update


def exec_plan(L: int, mask: Sequence[int]) -> Plan:
    """Section 2.2: a selected layer pays its own weight-gradient time, and every
    LATER layer pays its error-gradient time whether selected or not; nothing at or
    before the deepest selected layer passes a gradient further down."""
    mask = np.asarray(mask).astype(bool)
    assert mask.shape == (2 * L,)
    sel_layers = [l for l in range(L) if mask[2 * l] or mask[2 * l + 1]]
    d = min(sel_layers) if sel_layers else L
    return Plan(
        deepest=d,
        dgrad=np.array([l > d for l in range(L)]),
        wgrad=np.array([bool(mask[2 * l]) for l in range(L)]),
        bgrad=np.array([bool(mask[2 * l + 1]) for l in range(L)]),
        updated=mask.copy(),
    )


def executed_flops(layers, M: int, plan: Plan) -> float:
    """2*M*K*N per executed GEMM (dgrad and wgrad of one layer cost the same);
    normalisation layers are not GEMMs and count nothing."""
    fl = 0.0
    for l, ly in enumerate(layers):
        if _kind(ly) != KIND_DENSE:
            continue
        g = 2.0 * M * ly.in_features * ly.out_features
        fl += g * (int(plan.dgrad[l]) + int(plan.wgrad[l]))
    return fl


# --------------------------------------------------------------------------- backward
def _backward_sweep(layers, W, saved: Saved, dY: np.ndarray, stop: int,
                    want_w, want_b) -> Dict[int, np.ndarray]:
    """Reverse sweep over layers L-1 ... stop.  G[i] accumulates dL/da_i."""
    L = len(layers)
    G: List[Optional[np.ndarray]] = [None] * (L + 1)
    G[L] = np.asarray(dY, dtype=np.float64)
    grads: Dict[int, np.ndarray] = {}
    for l in range(L - 1, stop - 1, -1):
        ly = layers[l]
        g_out = G[l + 1]
        if _kind(ly) == KIND_BATCHNORM:
            xhat, rstd, z = saved.Z[l]
            dz = g_out * act_derivative(z, ly.act)
            if want_w[l]:
                grads[2 * l] = (dz * xhat).sum(axis=0)              # d gamma
            if want_b[l]:
                grads[2 * l + 1] = dz.sum(axis=0)                   # d beta
            if l > stop:
                # as for the row-wise normalisation, with the means taken over the rows of each column
                gy = dz * np.asarray(W[l], dtype=np.float64)
                dX = rstd * (gy - gy.mean(axis=0, keepdims=True) - xhat * (gy * xhat).mean(axis=0, keepdims=True))
                G[l] = dX if G[l] is None else G[l] + dX
            continue
        if _kind(ly) == KIND_IM2COL:
            if want_w[l]:
                grads[2 * l] = np.zeros(0)
            if want_b[l]:
                grads[2 * l + 1] = np.zeros(0)
            if l > stop:
                # every input pixel collects the gradient of each patch position it was copied to
                C_, Hh, Ww, k = ly.in_features, ly.height, ly.width, ly.ksize
                pd = k // 2
                gc = g_out.reshape(-1, Hh, Ww, k * k, C_)
                gp = np.zeros((gc.shape[0], Hh + 2 * pd, Ww + 2 * pd, C_))
                for kh in range(k):
                    for kw in range(k):
                        gp[:, kh:kh + Hh, kw:kw + Ww, :] += gc[:, :, :, kh * k + kw, :]
                dX = gp[:, pd:pd + Hh, pd:pd + Ww, :].reshape(-1, C_)
                G[l] = dX if G[l] is None else G[l] + dX
            continue
        if _kind(ly) == KIND_ATTENTION:
            if want_w[l]:
                grads[2 * l] = np.zeros(0)                                  # its tensor slots are empty
            if want_b[l]:
                grads[2 * l + 1] = np.zeros(0)
            if l > stop:
                P, q, k, v = saved.Z[l]
                B, H, S, dh = q.shape
                d = H * dh
                go = g_out.reshape(B, S, H, dh).transpose(0, 2, 1, 3)       # gradient of o, per head
                dv = P.transpose(0, 1, 3, 2) @ go
                dP = go @ v.transpose(0, 1, 3, 2)
                # softmax: dS_ij = P_ij (dP_ij - sum_j' P_ij' dP_ij')
                dS = P * (dP - (P * dP).sum(axis=-1, keepdims=True)) / np.sqrt(dh)
                dq = dS @ k
                dk = dS.transpose(0, 1, 3, 2) @ q
                dX = np.concatenate([t.transpose(0, 2, 1, 3).reshape(B * S, d) for t in (dq, dk, dv)], axis=1)
                G[l] = dX if G[l] is None else G[l] + dX
            continue
        if _kind(ly) == KIND_NORM:
            xhat, rstd = saved.Z[l]
            if want_w[l]:
                grads[2 * l] = (g_out * xhat).sum(axis=0)           # d gamma
            if want_b[l]:
                grads[2 * l + 1] = g_out.sum(axis=0)                # d beta
            if l > stop:
                # y = xhat*gamma + beta with xhat = (x - mean(x)) * rstd(x): differentiating through
                # the row mean and the row variance leaves the part of gy = g*gamma that is
                # orthogonal to the all-ones vector and to xhat, scaled by rstd
                gy = g_out * np.asarray(W[l], dtype=np.float64)
                dX = rstd * (gy - gy.mean(axis=1, keepdims=True)
                             - xhat * (gy * xhat).mean(axis=1, keepdims=True))
                G[l] = dX if G[l] is None else G[l] + dX
            continue
        if ly.residual_src >= 0:
            j = ly.residual_src
            G[j] = g_out.copy() if G[j] is None else G[j] + g_out
        # gradient w.r.t. H_l: each of the `fold` slices receives g_out
        dH = np.concatenate([g_out] * ly.fold, axis=1)
        dZ = dH * act_derivative(saved.Z[l], ly.act)
        if want_w[l]:
            grads[2 * l] = saved.a[l].T @ dZ                    # dW = X^T dZ
        if want_b[l]:
            grads[2 * l + 1] = dZ.sum(axis=0)                   # db = column sums
        if l > stop:
            dX = dZ @ np.asarray(W[l], dtype=np.float64).T      # dX = dZ W^T
            G[l] = dX if G[l] is None else G[l] + dX
    return grads


def backward_masked(layers, W, saved: Saved, dY: np.ndarray, mask):
    """Elastic backward: the sweep stops at the deepest selected layer, kernel /
    bias gradients are formed only for selected tensors."""
    L = len(layers)
    plan = exec_plan(L, mask)
    if plan.deepest == L:
        return {}, plan
    grads = _backward_sweep(layers, W, saved, dY, plan.deepest, plan.wgrad, plan.bgrad)
    return grads, plan


def backward_full(layers, W, saved: Saved, dY: np.ndarray) -> Dict[int, np.ndarray]:
    """Plain full backprop: every gradient of every tensor."""
    L = len(layers)
    return _backward_sweep(layers, W, saved, dY, 0, [True] * L, [True] * L)


# --------------------------------------------------------------------------- importance, update
def importance(grads: Dict[int, np.ndarray], delta: Sequence[np.ndarray], mask) -> np.ndarray:
    """Eq. (2): S_k = sum_i (dL/dw_i^k) * (delta w_i^k), for every selected tensor k;
    0 for the others."""
    out = np.zeros(len(mask))
    for k, m in enumerate(mask):
        if m:
            out[k] = float(np.sum(grads[k] * np.asarray(delta[k], dtype=np.float64)))
    return out


def magnitude_metric(tensors: Sequence[np.ndarray], mask) -> np.ndarray:
    """The non-additive metrics of the paper's ablation (Section 8, importance evaluator): the paper
    names them (weight magnitudes, gradient feedback) without a formula; read here as the L1 norm
    sum_i |x_i| of each selected tensor -- its weights for the first, its gradient for the second;
    0 for the others.  Unpinned against the paper (it prints no values); the tests pin it to the
    definition on hand-written vectors."""
    out = np.zeros(len(mask))
    for k, m in enumerate(mask):
        if m:
            out[k] = float(np.sum(np.abs(np.asarray(tensors[k], dtype=np.float64))))
    return out


def sgd_masked(params: Sequence[np.ndarray], grads: Dict[int, np.ndarray], mask, lr: float):
    """w <- w - lr * g for selected tensors; the others are returned untouched
    (same object, so a caller can check they were not rewritten)."""
    out = []
    for k, p in enumerate(params):
        out.append(p - lr * grads[k] if mask[k] else p)
    return out


def tensors_of(W, b):
    """Interleave kernels and biases into tensor order [W_0, b_0, W_1, b_1, ...]."""
    out = []
    for w_, b_ in zip(W, b):
        out += [w_, b_]
    return out


# --------------------------------------------------------------------------- time model, selector
def f_mask(mask) -> np.ndarray:
    """Eq. (3): f(M) marks every tensor whose error-gradient time is paid; for any
    selected tensor all later ones are included (and, in the example the paper
    prints, the selected one itself)."""
    m = np.asarray(mask).astype(bool)
    return np.logical_or.accumulate(m).astype(np.uint8)


def t_selective(mask, t_dw, t_dy, variant: int = STRICT) -> float:
    """Backward time of a selection.  STRICT follows the Section 2.2 example and
    Eq. (7): only tensors AFTER the deepest selected one pay t_dy.  INCLUSIVE is the
    f(M) of the Eq. (3) example, where the deepest selected tensor pays it too."""
    m = np.asarray(mask).astype(bool)
    t_dw = np.asarray(t_dw, dtype=np.float64)
    t_dy = np.asarray(t_dy, dtype=np.float64)
    if not m.any():
        return 0.0
    f = f_mask(m).astype(bool)
    if variant == STRICT:
        f = f.copy()
        f[int(np.argmax(m))] = False
    return float(t_dw[m].sum() + t_dy[f].sum())


def quantise(t_dw, t_dy, t_fwd: float, rho: float, Tq: int):
    """Eq. (8): t~ = floor(t * Z), Z = Tq / T with T the full backward time.  The
    budget for the backward pass is rho * T_full - T_fwd, T_full = T_fwd + T,
    floored the same way."""
    t_dw = np.asarray(t_dw, dtype=np.float64)
    t_dy = np.asarray(t_dy, dtype=np.float64)
    T = float(t_dw.sum() + t_dy.sum())
    Z = Tq / T
    qw = np.floor(t_dw * Z).astype(np.int64)
    qy = np.floor(t_dy * Z).astype(np.int64)
    budget = int(np.floor((rho * (t_fwd + T) - t_fwd) * Z))
    return qw, qy, budget


def select_bruteforce(I, qw, qy, budget: int, variant: int = STRICT):
    """Enumerate all 2^n masks of the integer-cost problem
    max M.I  s.t.  M.t_dw + f(M).t_dy <= budget   (Eq. 3 without the constant T_fwd)."""
    I = np.asarray(I, dtype=np.float64)
    n = len(I)
    best_val, best_mask = 0.0, np.zeros(n, dtype=np.uint8)
    for code in range(1, 1 << n):
        m = np.array([(code >> i) & 1 for i in range(n)], dtype=np.uint8)
        if t_selective(m, qw, qy, variant) <= budget:
            v = float(I[m.astype(bool)].sum())
            if v > best_val:
                best_val, best_mask = v, m
    return best_mask, best_val


def select_by_depth_knapsack(I, qw, qy, budget: int, variant: int = STRICT) -> float:
    """Second, independent route to the optimum: fix the deepest selected tensor d
    (it must be selected and fixes all t_dy charges), then the rest is a 0/1
    knapsack on t_dw over the tensors after d."""
    I = np.asarray(I, dtype=np.float64)
    n = len(I)
    best = 0.0
    for d in range(n):
        fixed = qw[d] + qy[d + 1:].sum() + (qy[d] if variant == INCLUSIVE else 0)
        cap = budget - fixed
        if cap < 0:
            continue
        knap = np.zeros(cap + 1)
        for i in range(d + 1, n):
            if I[i] <= 0:
                continue
            w = int(qw[i])
            if w == 0:
                knap = knap + I[i]
            elif w <= cap:
                knap[w:] = np.maximum(knap[w:], knap[:-w] + I[i])
        best = max(best, I[d] + knap[cap])
    return float(best)


def select_depth_knapsack_mask(I, qw, qy, budget: int, variant: int = STRICT):
    """Optimum AND a mask attaining it, for instances too large to enumerate: for every
    candidate deepest tensor d (selected by definition) a 0/1 knapsack with back-pointers over
    the tensors after d.  Used by the training-schedule oracle; checked against brute force."""
    I = np.asarray(I, dtype=np.float64)
    qw = np.asarray(qw, dtype=np.int64)
    qy = np.asarray(qy, dtype=np.int64)
    n = len(I)
    best_val, best_mask = 0.0, np.zeros(n, dtype=np.uint8)
    for d in range(n):
        fixed = int(qw[d] + qy[d + 1:].sum() + (qy[d] if variant == INCLUSIVE else 0))
        cap = budget - fixed
        if cap < 0:
            continue
        items = [i for i in range(d + 1, n) if I[i] > 0]
        table = np.zeros((len(items) + 1, cap + 1))
        for r, i in enumerate(items):
            w = int(qw[i])
            table[r + 1] = table[r]
            if w <= cap:
                cand = np.full(cap + 1, -np.inf)
                cand[w:] = table[r][:cap + 1 - w] + I[i]
                table[r + 1] = np.maximum(table[r], cand)
        val = I[d] + table[len(items)][cap]
        if val > best_val:
            mask = np.zeros(n, dtype=np.uint8)
            mask[d] = 1
            c = cap
            for r in range(len(items), 0, -1):
                if table[r][c] != table[r - 1][c]:
                    i = items[r - 1]
                    mask[i] = 1
                    c -= int(qw[i])
            best_val, best_mask = float(val), mask
    return best_mask, best_val


def train_schedule(layers, W, b, x, target, lr: float, steps: int, period: int, window: int,
                   rho: float, t_dw, t_dy, t_fwd: float = 0.0, Tq: int = 1000, variant: int = STRICT):
    """Elastic training schedule (Section 3.1): each period of `period` steps starts with
    `window` steps in which every tensor is trained; the weight change accumulated over the
    window, measured at the window's last step before that step's own update, gives the
    importances S_k = sum g * (w_now - w_window_start) of Eq. (2); -S_k (a loss decrease counts as
    positive, Section 4) goes to the selector at budget rho; the remaining steps of the period
    train the selected tensors only.  Plain SGD, one fixed batch.
    Returns per-step losses, per-step masks and the importances of every evaluation."""
    L = len(layers)
    W = [np.array(w_, dtype=np.float64) for w_ in W]
    b = [np.array(b_, dtype=np.float64) for b_ in b]
    losses, masks, evaluations = [], [], []
    mask = np.ones(2 * L, dtype=np.uint8)
    qw, qy, budget = quantise(t_dw, t_dy, t_fwd, rho, Tq)
    snap = None
    for step in range(steps):
        phase = step % period
        if phase == 0:
            mask = np.ones(2 * L, dtype=np.uint8)
            snap = [p.copy() for p in tensors_of(W, b)]
        saved = forward(layers, W, b, x)
        loss, dY = mse_loss_grad(saved.a[-1], target)
        grads, _ = backward_masked(layers, W, saved, dY, mask)
        losses.append(loss)
        masks.append(mask.copy())
        params = tensors_of(W, b)
        new_mask = None
        if phase == window - 1:
            delta = [p - s for p, s in zip(params, snap)]
            S = importance(grads, delta, mask)
            evaluations.append(S)
            new_mask, _ = select_depth_knapsack_mask(-S, qw, qy, budget, variant)
        new = sgd_masked(params, grads, mask, lr)
        W, b = list(new[0::2]), list(new[1::2])
        if new_mask is not None:
            mask = new_mask
    return dict(losses=np.array(losses), masks=masks, importances=evaluations, W=W, b=b)


# --------------------------------------------------------------------------- the paper's optimisers, masked
# Section 8: SGDW (momentum 0.9, decoupled weight decay 5e-4, cosine-scheduled learning rate) for the
# convolutional models and Adam (learning rate 1e-4) for ViT.  Only selected tensors (and their
# optimiser state) are touched.  The schedule lives with the caller: `lr` and `wd` are the values
# of the current step.
OPT_SGD, OPT_SGDW, OPT_ADAM = 0, 1, 2


def optimizer_state(params):
    """Zero-initialised state: first and second moment per tensor."""
    return [np.zeros_like(p, dtype=np.float64) for p in params], [np.zeros_like(p, dtype=np.float64) for p in params]


def optimizer_step_masked(params, grads, mask, kind, lr, state, step=1, momentum=0.9, wd=0.0,
                          beta1=0.9, beta2=0.999, eps=1e-8):
    """One masked update.  state = (m, v) lists as from optimizer_state, updated in place for
    selected tensors; returns the new parameter list (unselected entries are the same objects).
    SGDW (decoupled weight decay, Loshchilov & Hutter): m <- momentum*m + lr*g ;
        w <- w - m - wd*w  (decay applied to the old weight, not through the gradient).
    Adam (Kingma & Ba): m <- b1 m + (1-b1) g ; v <- b2 v + (1-b2) g^2 ;
        w <- w - lr * (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps),  t = step (1-based)."""
    m, v = state
    out = []
    for k, p in enumerate(params):
        if not mask[k]:
            out.append(p)
            continue
        g = grads[k]
        if kind == OPT_SGD:
            out.append(p - lr * g)
        elif kind == OPT_SGDW:
            m[k] = momentum * m[k] + lr * g
            out.append(p - m[k] - wd * p)
        elif kind == OPT_ADAM:
            m[k] = beta1 * m[k] + (1.0 - beta1) * g
            v[k] = beta2 * v[k] + (1.0 - beta2) * g * g
            mhat = m[k] / (1.0 - beta1 ** step)
            vhat = v[k] / (1.0 - beta2 ** step)
            out.append(p - lr * mhat / (np.sqrt(vhat) + eps))
        else:
            raise ValueError(kind)
    return out
