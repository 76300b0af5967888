"""Driver of the elastic training schedule over the C ABI (Section 3.1 of the paper):
periods that open with a window of all-tensor steps, an importance evaluation at the end of
the window, a re-selection by the host selector, then masked steps.

Control flow and marshalling only: every tensor operation is a library call
(et_forward_stack, et_loss_mse_grad, et_backward_elastic with the fused importance / SGD
epilogues, et_select_dp); torch is used for device buffers, snapshots (plain copies) and events.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as et


class ElasticLoop:
    def __init__(self, stack, W, b, x, target, lr, period, window, rho, t_dw, t_dy, t_fwd=0.0, Tq=1000,
                 variant=et.ET_COST_STRICT, stream=None, master=False):
        self.stack, self.W, self.b, self.x, self.target = stack, W, b, x, target
        self.lr, self.period, self.window, self.rho = float(lr), int(period), int(window), float(rho)
        self.t_dw, self.t_dy, self.t_fwd, self.Tq, self.variant = t_dw, t_dy, float(t_fwd), int(Tq), variant
        self.stream = stream
        self.L = stack.L
        dev = x.device
        self.y = torch.empty((stack.M, stack.out_width), dtype=x.dtype, device=dev)
        self.dY = torch.empty_like(self.y)
        self.params = [t for pair in zip(W, b) for t in pair]
        # master=True: fp32 master copies of bf16 parameters; updates and snapshots then live in fp32
        self.master = None
        if master:
            self.W32 = [t.float() for t in W]
            self.b32 = [t.float() for t in b]
            et.et_stack_bind_master(stack, self.W32, self.b32)
            self.master = [t for pair in zip(self.W32, self.b32) for t in pair]
        self.snap = [torch.empty_like(p) for p in (self.master or self.params)]
        self.imp = torch.zeros(2 * self.L, dtype=torch.float32, device=dev)
        # layers without tensors (attention core, patch gather) hold empty slots that cannot be selected
        self.all_mask = np.array([1 if p.numel() > 0 else 0 for p in self.params], dtype=np.uint8)
        self.mask = self.all_mask.copy()

    def run(self, steps, elastic=True, time_steps=False):
        """Runs `steps` training steps.  elastic=False trains every tensor at every step (full
        backprop, no evaluation).  Returns losses, the mask used at each step, the importances
        of each evaluation and, with time_steps, the mean device time per step in ms."""
        losses = torch.zeros(steps, dtype=torch.float32, device=self.x.device)
        masks, evaluations, dp_ms = [], [], []
        e0 = e1 = None
        if time_steps:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
        flags = et.ET_FLAG_FUSE_SGD
        for step in range(steps):
            phase = step % self.period
            if elastic and phase == 0:
                self.mask = self.all_mask.copy()
                for s_, p_ in zip(self.snap, self.master or self.params):
                    s_.copy_(p_)
            et.et_forward_stack(self.stack, self.x, self.y, stream=self.stream)
            et.et_loss_mse_grad(self.stack, self.y, self.target, self.dY, losses[step:step + 1], stream=self.stream)
            masks.append(self.mask.copy())
            if elastic and phase == self.window - 1:
                et.et_backward_elastic(self.stack, self.dY, self.mask, None, self.snap, self.imp,
                                       flags | et.ET_FLAG_DELTA_IS_SNAPSHOT, self.lr, None, stream=self.stream)
                S = self.imp.cpu().numpy().astype(np.float64)          # synchronises
                S = np.nan_to_num(S, nan=0.0, posinf=0.0, neginf=0.0)  # a diverged run must not stop the selector
                evaluations.append(S)
                import time
                t0 = time.perf_counter()
                self.mask, _, _ = et.et_select_dp(-S * self.all_mask, self.t_dw, self.t_dy, self.t_fwd, self.rho, self.Tq,
                                                  self.variant)
                self.mask = self.mask & self.all_mask
                dp_ms.append(1e3 * (time.perf_counter() - t0))
            else:
                et.et_backward_elastic(self.stack, self.dY, self.mask, None, None, None, flags, self.lr, None,
                                       stream=self.stream)
        out = dict(masks=masks, importances=evaluations, dp_ms=dp_ms)
        if time_steps:
            e1.record(self.stream)
            torch.cuda.synchronize()
            out["ms_per_step"] = e0.elapsed_time(e1) / steps
        out["losses"] = losses.cpu().numpy().astype(np.float64)
        return out

