"""Masked SGDW and Adam (the paper's optimisers, Section 8) through the C ABI against the oracle:
several consecutive training steps with the update fused into the backward call, and the
stand-alone update on exported gradients."""
import numpy as np
import pytest
import torch

import paper_2312_14227_b200 as et
import workloads as wl
from oracle import elastic_oracle as orc

pytestmark = pytest.mark.gpu

KINDS = {"sgdw": (orc.OPT_SGDW, et.ET_OPT_SGDW), "adam": (orc.OPT_ADAM, et.ET_OPT_ADAM)}


def _oracle_steps(w, mask, kind, lr, steps, wd_of_step, **kw):
    W, b = [a.copy() for a in w.W], [a.copy() for a in w.b]
    state = orc.optimizer_state(orc.tensors_of(W, b))
    losses = []
    for t in range(1, steps + 1):
        saved = orc.forward(w.layers, W, b, w.x)
        loss, dY = orc.mse_loss_grad(saved.a[-1], w.target)
        grads, _ = orc.backward_masked(w.layers, W, saved, dY, mask)
        new = orc.optimizer_step_masked(orc.tensors_of(W, b), grads, mask, kind, lr, state, step=t,
                                        wd=wd_of_step(t), **kw)
        W, b = list(new[0::2]), list(new[1::2])
        losses.append(loss)
    return W, b, state, np.array(losses)


@pytest.mark.parametrize("name", ["sgdw", "adam"])
@pytest.mark.parametrize("dtype", [wl.DT_F32, wl.DT_BF16])
def test_fused_optimizer_steps_match_oracle(name, dtype):
    import gpu_harness as h
    okind, gkind = KINDS[name]
    bf16 = dtype == wl.DT_BF16
    layers = wl.vit_blocks(1, 256, 512) if bf16 else wl.vit_blocks(1, 24, 40)
    rng = np.random.default_rng(3)
    mask = (rng.random(2 * len(layers)) < 0.6).astype(np.uint8)
    mask[0] = 1
    w = wl.small_stack(layers, 300 if bf16 else 50, dtype, 31, mask=mask, w_std=0.05, bias_std=0.02)
    steps = 4
    lr = 1e-3 if name == "adam" else 0.05
    wd = (lambda t: 5e-4 * (0.5 + 0.5 * np.cos(np.pi * t / 8))) if name == "sgdw" else (lambda t: 0.0)
    kw = dict(momentum=0.9) if name == "sgdw" else dict(beta1=0.9, beta2=0.999, eps=1e-8)
    W_ref, b_ref, st_ref, loss_ref = _oracle_steps(w, mask, okind, lr, steps, wd, **kw)

    run = h.GpuRun(w)
    params = run.params()
    master = None
    if bf16:
        W32, b32 = [t.float() for t in run.W], [t.float() for t in run.b]
        et.et_stack_bind_master(run.stack, W32, b32)
        master = [t for pair in zip(W32, b32) for t in pair]
    st1 = [torch.zeros(p.shape, dtype=torch.float32, device=h.DEV) for p in params]
    st2 = [torch.zeros(p.shape, dtype=torch.float32, device=h.DEV) for p in params]
    et.et_stack_set_optimizer(run.stack, gkind, st1, st2 if name == "adam" else None, **kw)
    before = [p.clone() for p in params]
    losses = []
    for t in range(1, steps + 1):
        et.et_stack_set_optimizer_step(run.stack, t, wd(t))
        run.forward_loss()
        losses.append(float(run.loss.item()))
        run.backward(mask, None, None, flags=et.ET_FLAG_FUSE_SGD, lr=lr)
    tol = 2e-2 if bf16 else 2e-4
    np.testing.assert_allclose(losses, loss_ref, rtol=tol)
    ref = orc.tensors_of(W_ref, b_ref)
    for t in range(2 * w.L):
        cur = h.to_np((master or params)[t])
        if mask[t]:
            scale = np.abs(ref[t] - orc.tensors_of(w.W, w.b)[t]).max()          # size of the total update
            err = np.abs(cur - ref[t])
            if bf16 and name == "adam":
                # Adam divides by |g|-sized quantities: where a gradient entry is small against the
                # tensor's largest, a bf16-level error of the gradient (relative to that largest
                # entry) moves the normalised step by O(lr).  Entries with a sizeable second moment
                # are well conditioned and held to a tight bound; the rest to the step size itself.
                rms = np.sqrt(st_ref[1][t] / (1.0 - 0.999 ** steps))
                well = rms >= 0.25 * rms.max()
                assert well.any()
                assert err[well].max() <= 0.1 * scale, (t, err[well].max(), scale)
                assert err.max() <= 1.05 * steps * lr and err.mean() <= 0.1 * scale, (t, err.max(), err.mean())
                continue
            assert err.max() <= tol * scale + 1e-7, (t, err.max(), scale)
            assert np.abs(h.to_np(st1[t]) - st_ref[0][t]).max() <= tol * np.abs(st_ref[0][t]).max() + 1e-12
            if name == "adam":
                assert np.abs(h.to_np(st2[t]) - st_ref[1][t]).max() <= 2 * tol * np.abs(st_ref[1][t]).max() + 1e-18
        else:
            assert torch.equal(params[t], before[t])
            assert not st1[t].any() and not st2[t].any()                         # frozen tensors keep no state


def test_standalone_update_matches_fused_optimizer_fp32():
    import gpu_harness as h
    layers = wl.mlp_blocks(2, 16, 24, wl.ACT_RELU)
    mask = np.array([1, 1, 0, 0, 1, 0, 1, 1], dtype=np.uint8)
    w = wl.small_stack(layers, 33, wl.DT_F32, 5, mask=mask, w_std=0.2, bias_std=0.1)
    results = []
    for fused in (True, False):
        run = h.GpuRun(w)
        params = run.params()
        st1 = [torch.zeros(p.shape, dtype=torch.float32, device=h.DEV) for p in params]
        st2 = [torch.zeros(p.shape, dtype=torch.float32, device=h.DEV) for p in params]
        et.et_stack_set_optimizer(run.stack, et.ET_OPT_ADAM, st1, st2)
        for t in (1, 2):
            et.et_stack_set_optimizer_step(run.stack, t, 0.0)
            run.forward_loss()
            if fused:
                run.backward(mask, None, None, flags=et.ET_FLAG_FUSE_SGD, lr=1e-2)
            else:
                grads = run.alloc_grads(mask)
                run.backward(mask, grads, None)
                et.et_update_masked(run.stack, mask, grads, 1e-2)
        torch.cuda.synchronize()
        results.append([p.clone() for p in params])
    for a, b in zip(*results):
        assert torch.equal(a, b)
