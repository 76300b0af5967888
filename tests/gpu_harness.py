"""Runs one workload through the CUDA library and through the oracle, for the parity tests.
Marshalling only: tensors are created from the shared seeded arrays, results are copied back."""
from __future__ import annotations

import numpy as np
import torch

import paper_2312_14227_b200 as et
import workloads as wl
from oracle import elastic_oracle as orc

DEV = "cuda:0"


def to_dev(a: np.ndarray, dtype: int) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    return t.to(torch.bfloat16 if dtype == wl.DT_BF16 else torch.float32).to(DEV).contiguous()


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


class GpuRun:
    """Holds device tensors of a workload bound to an et stack."""

    def __init__(self, w: wl.Workload):
        self.w = w
        self.stack = et.et_stack_create(w.layers, w.M, w.dtype)
        self.W = [to_dev(a, w.dtype) for a in w.W]
        self.b = [to_dev(a, w.dtype) for a in w.b]
        nbytes = et.et_stack_workspace_bytes(self.stack)
        self.ws = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
        assert self.ws.data_ptr() % 256 == 0
        et.et_stack_bind(self.stack, self.W, self.b, self.ws)
        self.x = to_dev(w.x, w.dtype)
        self.target = to_dev(w.target, w.dtype)
        tdt = torch.bfloat16 if w.dtype == wl.DT_BF16 else torch.float32
        self.y = torch.empty((w.M, w.layers[-1].out_width), dtype=tdt, device=DEV)
        self.dY = torch.empty_like(self.y)
        self.loss = torch.zeros(1, dtype=torch.float32, device=DEV)
        self.importance = torch.full((2 * w.L,), float("nan"), dtype=torch.float32, device=DEV)

    def params(self):
        out = []
        for W_, b_ in zip(self.W, self.b):
            out += [W_, b_]
        return out

    def forward_loss(self):
        et.et_forward_stack(self.stack, self.x, self.y)
        et.et_loss_mse_grad(self.stack, self.y, self.target, self.dY, self.loss)

    def alloc_grads(self, mask, sentinel=None):
        grads = []
        for t, p in enumerate(self.params()):
            if mask[t]:
                grads.append(torch.full(p.shape, float("nan"), dtype=torch.float32, device=DEV))
            else:
                grads.append(sentinel)
        return grads

    def backward(self, mask, grads=None, delta=None, flags=0, lr=0.0):
        rep = et.Report(self.w.L)
        et.et_backward_elastic(self.stack, self.dY, mask, grads, delta,
                               self.importance if delta is not None else None, flags, lr, rep)
        st = et.et_device_status(self.stack)
        assert st == et.ET_OK, et.et_status_string(st)
        return rep


def oracle_step(w: wl.Workload, mask, delta=None):
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    loss, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    grads, plan = orc.backward_masked(w.layers, w.W, saved, dY, mask)
    imp = orc.importance(grads, delta, mask) if delta is not None else None
    params = orc.tensors_of(w.W, w.b)
    new = orc.sgd_masked(params, grads, mask, w.lr)
    return dict(y=saved.a[-1], loss=loss, dY=dY, grads=grads, plan=plan, importance=imp, new=new, params=params)


def rel_max(a: np.ndarray, o: np.ndarray) -> float:
    """max-norm error relative to the max-norm of the oracle's tensor."""
    denom = float(np.abs(o).max())
    if denom == 0.0:
        return float(np.abs(a).max())
    return float(np.abs(a - o).max()) / denom


def importance_err(s_gpu: float, g: np.ndarray, d: np.ndarray) -> float:
    """Error of an importance sum relative to max(|S|, ||g||_inf * ||dw||_2).  The second
    term is the size of the error that gradient entries which are each off by
    tol * ||g||_inf, independently, put into the sum; it only matters when the terms of
    the sum cancel (a dw unrelated to g)."""
    s_o = float(np.sum(g * d))
    floor = float(np.abs(g).max()) * float(np.sqrt(np.sum(d * d)))
    return abs(s_gpu - s_o) / max(abs(s_o), floor, 1e-300)


def gradient_step_delta(w: wl.Workload, mask):
    """dw = -c * g with the oracle's own gradient (the update a gradient step makes), scaled
    to about 1e-3 and rounded to the storage type: the terms of the importance sum then all
    have one sign, so its plain relative error is meaningful."""
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    grads, _ = orc.backward_masked(w.layers, w.W, saved, dY, mask)
    rnd = wl.round_to_bf16 if w.dtype == wl.DT_BF16 else wl.round_to_f32
    out = wl.draw_delta(w, 0)
    for t, g in grads.items():
        m = float(np.abs(g).max())
        out[t] = rnd(-(1e-3 / m) * g) if m > 0 else np.zeros_like(g)
    return out


def check_step(w: wl.Workload, mask, tol: float, delta_seed: int = 77, w_tol: float = 1e-3, stats=None,
               aligned_delta: bool = False, derived_w_tol: bool = False):
    """Full parity check of one training step: forward, loss, elastic backward with fused
    importance and SGD.  Returns the report.  With aligned_delta the importance is checked
    by its plain relative error.  Updated weights must be within w_tol (1e-3) of the oracle's;
    with derived_w_tol the bound also admits what the arithmetic cannot avoid when weights or
    gradients are large: the bf16 store's half ulp (2^-9 |w|) and lr * tol * ||g||_inf from the
    gradient's own tolerance."""
    mask = np.asarray(mask, dtype=np.uint8)
    delta_np = gradient_step_delta(w, mask) if aligned_delta else wl.draw_delta(w, delta_seed)
    ref = oracle_step(w, mask, delta_np)
    run = GpuRun(w)
    before = [p.clone() for p in run.params()]
    run.forward_loss()
    assert rel_max(to_np(run.y), ref["y"]) <= tol
    assert abs(float(run.loss.item()) - ref["loss"]) <= tol * abs(ref["loss"])
    assert rel_max(to_np(run.dY), ref["dY"]) <= tol

    delta = [to_dev(d, w.dtype) for d in delta_np]
    grads = run.alloc_grads(mask)
    rep = run.backward(mask, grads, delta, flags=et.ET_FLAG_FUSE_SGD, lr=w.lr)

    plan = ref["plan"]
    assert rep.deepest == plan.deepest
    assert np.array_equal(rep.dgrad.astype(bool), plan.dgrad)
    assert np.array_equal(rep.wgrad.astype(bool), plan.wgrad)
    assert np.array_equal(rep.bgrad.astype(bool), plan.bgrad)
    assert np.array_equal(rep.updated.astype(bool), plan.updated)
    assert rep.flops_executed == orc.executed_flops(w.layers, w.M, plan)

    imp = to_np(run.importance)
    worst = 0.0
    # largest gradient entry of the step: the yardstick for gradients that are identically zero (a bias or
    # beta whose only effect is a per-column shift that a batch normalisation above removes again): the
    # oracle returns float64 noise for them, and "relative to the tensor's own largest entry" means nothing
    gscale = max([float(np.abs(ref["grads"][t]).max()) for t in range(2 * w.L) if mask[t] and ref["grads"][t].size] + [0.0])
    for t in range(2 * w.L):
        if mask[t]:
            g = to_np(grads[t])
            if g.size and float(np.abs(ref["grads"][t]).max()) < 1e-9 * gscale:
                assert float(np.abs(g).max()) <= tol * gscale, (t, "zero gradient", float(np.abs(g).max()))
                assert abs(imp[t]) <= tol * gscale * float(np.sqrt(np.sum(delta_np[t] ** 2))) + 1e-30
                assert np.all(np.abs(to_np(run.params()[t]) - ref["new"][t]) <= w_tol + 2.0 ** -8 * np.abs(ref["new"][t]))
                continue
            e = rel_max(g, ref["grads"][t])
            worst = max(worst, e)
            assert e <= tol, (t, e)
            ie = importance_err(imp[t], ref["grads"][t], delta_np[t])
            assert ie <= tol, (t, ie, imp[t])
            if aligned_delta and ref["importance"][t] != 0.0:
                assert abs(imp[t] - ref["importance"][t]) <= tol * abs(ref["importance"][t]), t
            new = to_np(run.params()[t])
            bound = w_tol
            if derived_w_tol:
                half_ulp = 2.0 ** -9 * np.abs(ref["new"][t]) if w.dtype == wl.DT_BF16 else 0.0
                bound = w_tol + half_ulp + w.lr * tol * float(np.abs(ref["grads"][t]).max())
            assert np.all(np.abs(new - ref["new"][t]) <= bound), t
        else:
            assert imp[t] == 0.0
            assert torch.equal(run.params()[t], before[t]), f"frozen tensor {t} was written"
    if stats is not None:
        stats["worst_grad_rel"] = worst
    return rep
