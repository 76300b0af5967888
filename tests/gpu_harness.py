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

    def __init__(self, w: wl.Workload, gemm_list=None):
        """gemm_list: None = the library's default; False = one launch per GEMM (the two-stream path) even where
        the one-launch backward would apply; True = say so explicitly."""
        self.w = w
        et.et_debug_guard_regions(True)          # every test stack carries guard words round its workspace regions
        self.stack = et.et_stack_create(w.layers, w.M, w.dtype)
        et.et_debug_guard_regions(False)
        if gemm_list is not None:
            et.et_stack_set_option(self.stack, et.ET_OPTION_GEMM_LIST, 1 if gemm_list else 0)
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

    def check_guards(self):
        st, bad = et.et_debug_check_guards(self.stack)
        assert st == et.ET_OK, f"{et.et_status_string(st)} (region {bad})"

    def forward_loss(self):
        et.et_forward_stack(self.stack, self.x, self.y)
        et.et_loss_mse_grad(self.stack, self.y, self.target, self.dY, self.loss)
        self.check_guards()

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
        self.check_guards()
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


class StepChecker:
    """Parity checks of elastic steps on one workload, sharing what does not depend on the mask: the
    oracle's forward pass and loss gradient, the device buffers and the GPU's forward pass.  Each
    check() restores the parameters, runs one elastic backward with fused importance and SGD through
    the C ABI and compares everything with the oracle's masked backward for that mask.

    master=True attaches fp32 master copies of bf16 parameters (the update is applied to them and the
    bf16 tensors are rewritten as their roundings)."""

    def __init__(self, w: wl.Workload, tol: float, master: bool = False, gemm_list=None):
        self.w, self.tol, self.master = w, tol, master
        self.saved = orc.forward(w.layers, w.W, w.b, w.x)
        self.loss, self.dY = orc.mse_loss_grad(self.saved.a[-1], w.target)
        self.params_o = orc.tensors_of(w.W, w.b)
        self._grads = {}
        run = self.run = GpuRun(w, gemm_list=gemm_list)
        self.before = [p.clone() for p in run.params()]
        self.m32 = None
        if master:
            self.W32 = [t.float() for t in run.W]
            self.b32 = [t.float() for t in run.b]
            et.et_stack_bind_master(run.stack, self.W32, self.b32)
            self.m32 = [t for pair in zip(self.W32, self.b32) for t in pair]
        run.forward_loss()
        assert rel_max(to_np(run.y), self.saved.a[-1]) <= tol
        assert abs(float(run.loss.item()) - self.loss) <= tol * abs(self.loss)
        assert rel_max(to_np(run.dY), self.dY) <= tol

    def oracle_backward(self, mask):
        key = bytes(np.asarray(mask, dtype=np.uint8))
        if key not in self._grads:
            self._grads = {key: orc.backward_masked(self.w.layers, self.w.W, self.saved, self.dY, mask)}   # keep one
        return self._grads[key]

    def _restore(self):
        for p, q in zip(self.run.params(), self.before):
            p.copy_(q)
        if self.m32 is not None:
            for m, q in zip(self.m32, self.before):
                m.copy_(q)

    def check(self, mask, delta_seed: int = 77, w_tol: float = 1e-3, stats=None, aligned_delta: bool = False,
              derived_w_tol: bool = False, snapshot: bool = False):
        """aligned_delta: dw = -c * g with the oracle's own gradient, so that every term of the importance
        sum has one sign and its plain relative error must be within tol.  snapshot: the delta tensors hold
        a snapshot W - dw of the weights (ET_FLAG_DELTA_IS_SNAPSHOT; fp32 when master weights are attached)
        instead of dw itself.  stats (a dict) receives diagnostics: the worst max-norm gradient error, the
        worst plain relative importance error and the worst elementwise gradient error relative to
        max(|o|, 2^-6 ||o||_inf)."""
        w, tol, run = self.w, self.tol, self.run
        mask = np.asarray(mask, dtype=np.uint8)
        self._restore()
        g_o, plan = self.oracle_backward(mask)
        rnd = wl.round_to_bf16 if w.dtype == wl.DT_BF16 else wl.round_to_f32
        delta_np = wl.draw_delta(w, delta_seed if not aligned_delta else 0)
        if aligned_delta:
            for t, g in g_o.items():
                m = float(np.abs(g).max())
                delta_np[t] = rnd(-(1e-3 / m) * g) if m > 0 else np.zeros_like(g)
        flags = et.ET_FLAG_FUSE_SGD
        if snapshot:
            # what the library is given: the weights at the window start; what Eq. 2 then uses: W - snapshot
            rs = wl.round_to_f32 if (self.master or w.dtype != wl.DT_BF16) else wl.round_to_bf16
            snap_np = [rs(p - d) if p.size else p for p, d in zip(self.params_o, delta_np)]
            delta_np = [p - s for p, s in zip(self.params_o, snap_np)]
            if self.master:
                delta = [torch.from_numpy(np.ascontiguousarray(s)).to(torch.float32).to(DEV) for s in snap_np]
            else:
                delta = [to_dev(s, w.dtype) for s in snap_np]
            flags |= et.ET_FLAG_DELTA_IS_SNAPSHOT
        else:
            delta = [to_dev(d, w.dtype) for d in delta_np]
        imp_o = orc.importance(g_o, delta_np, mask)
        new_o = orc.sgd_masked(self.params_o, g_o, mask, w.lr)

        grads = run.alloc_grads(mask)
        run.importance.fill_(float("nan"))
        rep = run.backward(mask, grads, delta, flags=flags, lr=w.lr)

        assert rep.deepest == plan.deepest
        assert np.array_equal(rep.dgrad.astype(bool), plan.dgrad)
        assert np.array_equal(rep.wgrad.astype(bool), plan.wgrad)
        assert np.array_equal(rep.bgrad.astype(bool), plan.bgrad)
        assert np.array_equal(rep.updated.astype(bool), plan.updated)
        assert rep.flops_executed == orc.executed_flops(w.layers, w.M, plan)

        imp = to_np(run.importance)
        worst = worst_imp_rel = worst_elt = 0.0
        # largest gradient entry of the step: the yardstick for gradients that are identically zero (a bias or
        # beta whose only effect is a per-column shift that a batch normalisation above removes again): the
        # oracle returns float64 noise for them, and "relative to the tensor's own largest entry" means nothing
        gscale = max([float(np.abs(g_o[t]).max()) for t in range(2 * w.L) if mask[t] and g_o[t].size] + [0.0])
        live = self.m32 if self.m32 is not None else run.params()
        for t in range(2 * w.L):
            if mask[t]:
                g = to_np(grads[t])
                if g.size and float(np.abs(g_o[t]).max()) < 1e-9 * gscale:
                    assert float(np.abs(g).max()) <= tol * gscale, (t, "zero gradient", float(np.abs(g).max()))
                    assert abs(imp[t]) <= tol * gscale * float(np.sqrt(np.sum(delta_np[t] ** 2))) + 1e-30
                    assert np.all(np.abs(to_np(live[t]) - new_o[t]) <= w_tol + 2.0 ** -8 * np.abs(new_o[t]))
                    continue
                e = rel_max(g, g_o[t])
                worst = max(worst, e)
                assert e <= tol, (t, e)
                gmax = float(np.abs(g_o[t]).max())
                worst_elt = max(worst_elt, float((np.abs(g - g_o[t]) / np.maximum(np.abs(g_o[t]), 2.0 ** -6 * gmax)).max()))
                ie = importance_err(imp[t], g_o[t], delta_np[t])
                assert ie <= tol, (t, ie, imp[t])
                if imp_o[t] != 0.0:
                    plain = abs(imp[t] - imp_o[t]) / abs(imp_o[t])
                    worst_imp_rel = max(worst_imp_rel, plain)
                    if aligned_delta:
                        assert plain <= tol, (t, plain)
                new = to_np(live[t])
                bound = w_tol
                if derived_w_tol:
                    half_ulp = 2.0 ** -9 * np.abs(new_o[t]) if (w.dtype == wl.DT_BF16 and self.m32 is None) else 0.0
                    bound = w_tol + half_ulp + w.lr * tol * gmax
                assert np.all(np.abs(new - new_o[t]) <= bound), t
                if self.m32 is not None:      # the stored tensor is the rounding of its master
                    assert torch.equal(run.params()[t], self.m32[t].to(run.params()[t].dtype)), t
            else:
                assert imp[t] == 0.0
                assert torch.equal(run.params()[t], self.before[t]), f"frozen tensor {t} was written"
                if self.m32 is not None:
                    assert torch.equal(self.m32[t], self.before[t].float()), f"frozen master {t} was written"
        if stats is not None:
            stats["worst_grad_rel"] = max(worst, stats.get("worst_grad_rel", 0.0))
            stats["worst_grad_elementwise_rel_floor_2^-6"] = max(worst_elt, stats.get("worst_grad_elementwise_rel_floor_2^-6", 0.0))
            key = "worst_importance_plain_rel_" + ("aligned" if aligned_delta else "random")
            stats[key] = max(worst_imp_rel, stats.get(key, 0.0))
        return rep


def check_step(w: wl.Workload, mask, tol: float, delta_seed: int = 77, w_tol: float = 1e-3, stats=None,
               aligned_delta: bool = False, derived_w_tol: bool = False, gemm_list=None):
    """Full parity check of one training step: forward, loss, elastic backward with fused
    importance and SGD.  Returns the report.  With aligned_delta the importance is checked
    by its plain relative error.  Updated weights must be within w_tol (1e-3) of the oracle's;
    with derived_w_tol the bound also admits what the arithmetic cannot avoid when weights or
    gradients are large: the bf16 store's half ulp (2^-9 |w|) and lr * tol * ||g||_inf from the
    gradient's own tolerance."""
    return StepChecker(w, tol, gemm_list=gemm_list).check(mask, delta_seed=delta_seed, w_tol=w_tol, stats=stats,
                                                          aligned_delta=aligned_delta, derived_w_tol=derived_w_tol)
