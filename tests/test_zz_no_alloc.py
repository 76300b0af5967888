"""The allocation-free bias-gradient entry point against the ordinary one.

Some users of this library run where device memory may not be allocated at the moment a
bias gradient is needed (a plug-in inside an application that owns the GPU's memory, a
latency-critical callback, a fixed start-up budget), so et_bias_grad_noalloc keeps its
intermediate sums in an array built into the library.  This file is collected last on
purpose: a run that stops at the first failure has then already run everything else.
"""
import numpy as np
import pytest
import torch

import paper_2312_14227_b200 as et
import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _reference_bias_grad(dY: torch.Tensor, dtype: int) -> torch.Tensor:
    """db through the existing entry point: a one-layer stack whose only selected tensor is
    its bias, so et_backward_elastic runs exactly the bias gradient of dY."""
    M, width = dY.shape
    tdt = dY.dtype
    stack = et.et_stack_create([wl.Layer(width, width)], M, dtype)
    W = [torch.zeros((width, width), dtype=tdt, device=DEV)]
    b = [torch.zeros(width, dtype=tdt, device=DEV)]
    ws = torch.empty(et.et_stack_workspace_bytes(stack), dtype=torch.uint8, device=DEV)
    et.et_stack_bind(stack, W, b, ws)
    x = torch.zeros((M, width), dtype=tdt, device=DEV)
    y = torch.empty_like(x)
    et.et_forward_stack(stack, x, y)
    db = torch.full((width,), float("nan"), dtype=torch.float32, device=DEV)
    et.et_backward_elastic(stack, dY, np.array([0, 1], dtype=np.uint8), [None, db])
    torch.cuda.synchronize()
    return db


@pytest.mark.parametrize("dtype,tol", [(wl.DT_F32, 1e-4), (wl.DT_BF16, 2e-2)])
def test_noalloc_bias_grad_matches_existing_entry_point_twice(dtype, tol):
    tdt = torch.bfloat16 if dtype == wl.DT_BF16 else torch.float32
    gen = torch.Generator(device="cpu").manual_seed(1234 + dtype)
    # two calls in a row with different shapes and data: the second one finds the first
    # one's partial sums still in the built-in scratch and must not be affected by them
    for M, width in ((1000, 264), (333, 72)):
        dY = torch.randn((M, width), generator=gen).to(tdt).to(DEV).contiguous()
        want = _reference_bias_grad(dY, dtype)
        got = torch.full((width,), float("nan"), dtype=torch.float32, device=DEV)
        et.et_bias_grad_noalloc(dY, M, width, dtype, got)
        torch.cuda.synchronize()
        scale = float(want.abs().max())
        assert float((got - want).abs().max()) <= tol * scale
        # and against a direct sum, so that a fault shared by both entry points would show too
        direct = dY.double().sum(dim=0)
        assert float((got.double() - direct).abs().max()) <= tol * float(direct.abs().max())


def test_noalloc_rejects_sizes_beyond_the_builtin_scratch():
    width = 4096
    M = 128 * (et.ET_NOALLOC_SCRATCH_FLOATS // width) + 1          # one chunk too many
    dummy = torch.zeros(8, dtype=torch.float32, device=DEV)         # never dereferenced: the call is refused first
    with pytest.raises(et.EtError) as e:
        et.et_bias_grad_noalloc(dummy, M, width, wl.DT_F32, dummy)
    assert e.value.status == et.ET_ERR_TOO_LARGE
    with pytest.raises(et.EtError) as e:
        et.et_bias_grad_noalloc(dummy, 0, width, wl.DT_F32, dummy)
    assert e.value.status == et.ET_ERR_INVALID_ARG


@pytest.mark.parametrize("M,width", [(12608, 3072), (128 * 256, 4096)])
def test_noalloc_bias_grad_up_to_the_whole_scratch(M, width):
    # 99 and 256 chunks of partial sums: the finishing kernel's strided loop over more than 32 chunks, and
    # (second shape) a problem that fills the built-in array to its last float
    assert -(-M // 128) * width <= et.ET_NOALLOC_SCRATCH_FLOATS
    gen = torch.Generator(device="cpu").manual_seed(99)
    dY = torch.randn((M, width), generator=gen).to(torch.bfloat16).to(DEV).contiguous()
    got = torch.full((width,), float("nan"), dtype=torch.float32, device=DEV)
    et.et_bias_grad_noalloc(dY, M, width, wl.DT_BF16, got)
    torch.cuda.synchronize()
    direct = dY.double().sum(dim=0)
    assert float((got.double() - direct).abs().max()) <= 1e-4 * float(direct.abs().max())
    want = _reference_bias_grad(dY, wl.DT_BF16)
    assert float((got - want).abs().max()) <= 1e-5 * float(want.abs().max())
