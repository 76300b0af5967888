#!/usr/bin/env python
"""Benchmark of the elastic backward step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one pass of the hot path over one batch: the execution plan from the mask, the
error-gradient GEMMs above the deepest selected layer, the weight-gradient GEMMs, bias
gradients, importance reduction and masked SGD of the selected tensors.  The forward pass and
the loss gradient run once before the timed region (they precede the hot path).

Workload: the ViT-B/16-shaped linear-only stack (12 blocks, 64 x 197 tokens, bf16 storage with
fp32 accumulation, seeded Bernoulli(0.3) selection mask), synthetic N(0,1) inputs.
Metric: executed TFLOP/s of the elastic backward step (2*M*K*N per executed GEMM; work the
mask removes is not counted), with the step time beside it and the full-backprop step time
for comparison.

With --gpus N > 1 every rank runs an independent replica (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

METRIC = "elastic_backward_executed_tflops"
UNIT = "TFLOP/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


NOMINAL_BF16_TFLOPS = 2250.0      # dense bf16 tensor peak of the part, for context beside the measured peaks
NOMINAL_HBM_GBS = 8000.0


def tensor_fracs(tf: float, peaks: dict) -> dict:
    """One achieved TFLOP/s figure against the three denominators in use."""
    return {"of_measured_burst": tf / peaks["tf_burst"], "of_measured_sustained": tf / peaks["tf_sustained"],
            "of_nominal_dense": tf / NOMINAL_BF16_TFLOPS}


def _list_traffic(blocks: int):
    """DRAM bytes of one gemm_list_kernel launch from the committed ncu capture (taken on a reduced stack of the
    same shapes, scaled by executed flops), or None once the GEMM sources have changed since the counters were
    taken."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "gemm_list_dram_traffic.json")) as f:
            rec = json.load(f)
        h = hashlib.sha256()
        for name in ("gemm_tc.cuh", "gemm_list.cuh", "epilogue.cuh"):
            with open(os.path.join(ROOT, "paper_2312_14227_b200", "csrc", name), "rb") as f:
                h.update(f.read())
        if h.hexdigest() != rec["source_sha256"]:
            return None
        return rec["bytes_per_tflop"] * rec["tflop_of_benchmark_step"] if blocks == 12 else None
    except (OSError, KeyError, ValueError):
        return None


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------ reference arm
def oracle_sample(w_full: wl.Workload, n_blocks: int):
    """Bounded sample of the workload for the CPU oracle: the top n_blocks transformer blocks of
    the same stack (same widths, same token count, the mask bits of those layers)."""
    from oracle import elastic_oracle as orc
    layers = wl.vit_blocks(n_blocks, 768, 3072)
    L = len(layers)
    mask = w_full.mask[-2 * L:].copy()
    if not mask.any():
        mask[-2:] = 1
    w = wl.small_stack(layers, w_full.M, wl.DT_BF16, 123, mask=mask, w_std=0.02)
    saved = orc.forward(w.layers, w.W, w.b, w.x)
    _, dY = orc.mse_loss_grad(saved.a[-1], w.target)
    delta = wl.draw_delta(w, 5)
    params = orc.tensors_of(w.W, w.b)

    def step():
        t0 = time.perf_counter()
        grads, plan = orc.backward_masked(w.layers, w.W, saved, dY, mask)
        orc.importance(grads, delta, mask)
        orc.sgd_masked(params, grads, mask, w.lr)
        dt = time.perf_counter() - t0
        return dt, orc.executed_flops(w.layers, w.M, plan)

    return step, f"oracle masked backward + importance + SGD on the top {n_blocks} of 12 blocks, all {w.M} tokens, float64"


ORACLE_SAMPLE_BLOCKS = 1      # both the reference arm and the cpu_baseline leg time this sample


def time_oracle(w_full: wl.Workload, steps: int, warmup: int):
    """Times the oracle as it stands on the bounded sample: `warmup` untimed calls, then `steps` timed ones.
    Returns (list of seconds, executed flops per step, description of the sample)."""
    step, sample = oracle_sample(w_full, ORACLE_SAMPLE_BLOCKS)
    for _ in range(warmup):
        step()
    times, flops = [], 0.0
    for _ in range(steps):
        dt, flops = step()
        times.append(dt)
    sample += f" (the top {ORACLE_SAMPLE_BLOCKS} of 12 blocks with its own mask bits: about 1/12 of the configuration's work)"
    return times, flops, sample


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.vit_b(params=False)
    warm = max(1, min(args.warmup, 3))          # one block per step keeps K steps within minutes
    times, flops, sample = time_oracle(w, args.steps, warm)
    ms = 1e3 * float(np.mean(times))
    val = flops / (ms * 1e-3) / 1e12
    cores = blas_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "vit_b_linear_bf16 (oracle sample)", "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                         "median_value": flops / float(np.median(times)) / 1e12},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------ own arm
def max_over_ranks(ms: float, dist, device) -> float:
    """Step time of the job = the slowest rank's (every rank runs an independent replica)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(flops_per_rank: float, ms: float, world: int) -> float:
    """Whole-job executed TFLOP/s: all ranks' work over the slowest rank's time."""
    return world * flops_per_rank / (ms * 1e-3) / 1e12


def run_own(args):
    import torch
    import paper_2312_14227_b200 as et

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w = wl.vit_b() if args.blocks == 12 else wl.vit_b(n_blocks=args.blocks, name=f"vit_b_linear_bf16_{args.blocks}blocks")
    if args.profile:
        w.mask[:] = 1
    tdt = torch.bfloat16

    def to_dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(tdt).to(dev).contiguous()

    stack = et.et_stack_create(w.layers, w.M, w.dtype)
    if args.plain_launch:
        et.et_stack_set_option(stack, et.ET_OPTION_LIST_COOPERATIVE, 0)
    W = [to_dev(a) for a in w.W]
    b = [to_dev(a) for a in w.b]
    ws = torch.empty(et.et_stack_workspace_bytes(stack), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    et.et_stack_bind(stack, W, b, ws, stream=stream)
    x, target = to_dev(w.x), to_dev(w.target)
    y = torch.empty((w.M, w.layers[-1].out_width), dtype=tdt, device=dev)
    dY = torch.empty_like(y)
    delta = [to_dev(d) for d in wl.draw_delta(w, 5)]
    imp = torch.zeros(2 * w.L, dtype=torch.float32, device=dev)
    et.et_forward_stack(stack, x, y, stream=stream)
    et.et_loss_mse_grad(stack, y, target, dY, None, stream=stream)
    torch.cuda.synchronize()
    if args.optimizer != "sgd":                     # the paper's optimisers, with fp32 master weights
        W32, b32 = [t.float() for t in W], [t.float() for t in b]
        et.et_stack_bind_master(stack, W32, b32)
        params = [t for pair in zip(W, b) for t in pair]
        st1 = [torch.zeros(p.shape, dtype=torch.float32, device=dev) for p in params]
        st2 = [torch.zeros(p.shape, dtype=torch.float32, device=dev) for p in params]
        if args.optimizer == "sgdw":
            et.et_stack_set_optimizer(stack, et.ET_OPT_SGDW, st1, None, momentum=0.9, weight_decay=5e-4)
        else:
            et.et_stack_set_optimizer(stack, et.ET_OPT_ADAM, st1, st2)
    dY_host = dY.cpu().pin_memory()
    imp_host = torch.zeros(2 * w.L, dtype=torch.float32).pin_memory()
    ones = np.ones(2 * w.L, dtype=np.uint8)
    rep = et.Report(w.L)
    flags = et.ET_FLAG_FUSE_SGD

    def step(mask):
        et.et_backward_elastic(stack, dY, mask, None, delta, imp, flags, w.lr, rep, stream=stream)

    if args.profile:
        # short run for a profiler: forward above, then two full-backprop steps of a reduced stack
        step(w.mask)
        step(w.mask)
        torch.cuda.synchronize()
        assert et.et_device_status(stack, stream=stream) == et.ET_OK
        print(json.dumps({"profile_run": w.name, "launches": et.et_launch_count()}))
        return

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = et.et_launch_count()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        ms = max_over_ranks(e0.elapsed_time(e1) / steps, dist, dev)
        return ms, et.et_launch_count() - n0

    sampler = ClockSampler(local)
    sampler.start()
    # forward (context) and full backprop (comparison)
    fwd_ms, _ = timed(lambda: et.et_forward_stack(stack, x, y, stream=stream), max(2, args.steps // 4), 2)
    full_ms, _ = timed(lambda: step(ones), args.steps, args.warmup)
    full_flops = rep.flops_executed

    # the headline: elastic step, device-resident inputs
    ms, launches = timed(lambda: step(w.mask), args.steps, args.warmup)
    flops = rep.flops_executed
    st = et.et_device_status(stack, stream=stream)
    assert st == et.ET_OK, et.et_status_string(st)
    value = aggregate_value(flops, ms, world)

    # end to end through the host-buffer entry point: dY comes from pinned host memory and the
    # importances go back to it, inside the timed region
    def step_host():
        et.et_backward_elastic_host(stack, dY_host, w.mask, None, delta, imp_host, flags, w.lr, rep, stream=stream)

    e2e_ms, _ = timed(step_host, args.steps, args.warmup)
    e2e_value = aggregate_value(flops, e2e_ms, world)
    clocks = sampler.stop()     # sampled from the full-backprop run to the end of the end-to-end run

    # Device time per kernel class (a CUDA-event pair around every launch, recorded by the library on the
    # launching stream over the same steps).  The timed step above runs every GEMM of the pass in ONE
    # cooperative launch (gemm_list_kernel), followed by one grouped split reducer and one grouped bias
    # finisher: that launch is the dominant kernel.  For comparison the same step is also timed launched GEMM by
    # GEMM (the path stacks with other layer kinds take), as a two-stream step and class by class.
    peaks = _peaks()
    M = w.M
    first = next(l for l in range(w.L) if w.mask[2 * l] or w.mask[2 * l + 1])
    dgrad_flops = sum(2.0 * M * ly.in_features * ly.out_features for l, ly in enumerate(w.layers) if l > first)
    wgrad_flops = sum(2.0 * M * ly.in_features * ly.out_features for l, ly in enumerate(w.layers) if w.mask[2 * l])
    sel_params = sum(ly.in_features * ly.out_features for l, ly in enumerate(w.layers) if w.mask[2 * l])
    # bytes the reducer must move per selected kernel tensor of P parameters: 4P (gradient) + 2P (dW) + 2P + 2P
    # (W in / out); re-reading more than one split's partial sums is its own scratch traffic
    reduce_bytes = 10.0 * sel_params

    def classes_of(step_fn, n_steps):
        et.et_timing_enable(stack, True)
        inst_ms, _ = timed(step_fn, n_steps, 1)
        classes = et.et_timing_read(stack)
        et.et_timing_enable(stack, False)
        n_rec = n_steps + 1             # the warm-up step is in the record too: normalise by recorded steps
        return {k: (t / n_rec, n / n_rec) for k, (t, n) in classes.items()}, inst_ms

    def gb(ms_):
        return reduce_bytes / (ms_ * 1e-3) / 1e9 if ms_ > 0 else 0.0

    cls, inst_ms = classes_of(lambda: step(w.mask), args.steps)
    ls_ms, ls_n = cls["gemm_list"]
    ls_tf = flops / (ls_ms * 1e-3) / 1e12 if ls_ms > 0 else 0.0
    one_launch = {
        "gemm_list": {"launches_per_step": ls_n, "ms_per_step": ls_ms, "achieved": ls_tf, "unit": "TFLOP/s",
                      "flops_per_launch": flops, "frac": tensor_fracs(ls_tf, peaks),
                      "what": "all %d error-gradient and %d weight-gradient GEMMs of the step as work units of one "
                              "cooperative launch" % (int(rep.dgrad.sum()), int(rep.wgrad.sum()))},
        "wgrad_reduce_importance_sgd": {"launches_per_step": cls["wgrad_reduce"][1], "ms_per_step": cls["wgrad_reduce"][0],
                                        "achieved": gb(cls["wgrad_reduce"][0]), "unit": "GB/s",
                                        "algorithmic_bytes_per_step": reduce_bytes,
                                        "frac_of_hbm_peak": gb(cls["wgrad_reduce"][0]) / peaks["hbm_gbs"]},
        "bias_grad": {"launches_per_step": cls["bgrad"][1], "ms_per_step": cls["bgrad"][0],
                      "note": "top layer's column sums + one grouped finisher (the other column sums come out of the "
                              "error-gradient epilogues): a few MB of partials per step, reported as time"},
        "other": {"launches_per_step": cls["other"][1], "ms_per_step": cls["other"][0]},
        "instrumented_step_ms": inst_ms,
    }
    # the same step, one launch per GEMM
    et.et_stack_set_option(stack, et.ET_OPTION_GEMM_LIST, 0)
    pl_ms, pl_launches = timed(lambda: step(w.mask), args.steps, args.warmup)
    pl_full_ms, _ = timed(lambda: step(ones), max(2, args.steps // 4), 2)
    et.et_stack_set_option(stack, et.ET_OPTION_TILE_PLAN, et.ET_TILE_PLAN_SHARED)
    pcls, p_inst = classes_of(lambda: step(w.mask), max(2, args.steps // 4))
    et.et_stack_set_option(stack, et.ET_OPTION_TILE_PLAN, et.ET_TILE_PLAN_AUTO)
    et.et_stack_set_option(stack, et.ET_OPTION_GEMM_LIST, 1)
    dg_tf = dgrad_flops / (pcls["dgrad"][0] * 1e-3) / 1e12 if pcls["dgrad"][0] > 0 else 0.0
    wg_tf = wgrad_flops / (pcls["wgrad"][0] * 1e-3) / 1e12 if pcls["wgrad"][0] > 0 else 0.0
    per_layer = {
        "two_stream_step_ms": pl_ms, "two_stream_step_tflops": flops / (pl_ms * 1e-3) / 1e12,
        "two_stream_full_backprop_ms": pl_full_ms, "launches_per_step": pl_launches / args.steps,
        "dgrad_gemm": {"launches_per_step": pcls["dgrad"][1], "ms_per_step": pcls["dgrad"][0], "achieved": dg_tf,
                       "unit": "TFLOP/s", "frac": tensor_fracs(dg_tf, peaks)},
        "wgrad_gemm": {"launches_per_step": pcls["wgrad"][1], "ms_per_step": pcls["wgrad"][0], "achieved": wg_tf,
                       "unit": "TFLOP/s", "frac": tensor_fracs(wg_tf, peaks)},
        "wgrad_reduce_importance_sgd": {"launches_per_step": pcls["wgrad_reduce"][1], "ms_per_step": pcls["wgrad_reduce"][0],
                                        "achieved": gb(pcls["wgrad_reduce"][0]), "unit": "GB/s",
                                        "frac_of_hbm_peak": gb(pcls["wgrad_reduce"][0]) / peaks["hbm_gbs"]},
        "bias_grad": {"launches_per_step": pcls["bgrad"][1], "ms_per_step": pcls["bgrad"][0]},
        "note": "classes timed one kernel at a time on one stream (event pair per launch, which adds about 3 us to "
                "each), with the tile shapes the two-stream step launches",
    }
    kernels = {"one_launch": one_launch, "per_layer": per_layer}
    timed_span_s = ms * args.steps * 1e-3
    use_burst = timed_span_s < 1.0
    peak = peaks["tf_burst"] if use_burst else peaks["tf_sustained"]

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": w.name, "blocks": args.blocks, "tokens": w.M, "d": 768, "ffn": 3072,
                   "mask": "Bernoulli(0.3) per kernel tensor, seed 1, bias follows kernel",
                   "selected_tensors": int(w.mask.sum()), "deepest_selected_layer": first,
                   "step": "et_backward_elastic with fused importance and " + {"sgd": "SGD", "sgdw": "SGDW (fp32 master weights)", "adam": "Adam (fp32 master weights)"}[args.optimizer],
                   "l2": "inputs larger than L2 (a step streams > 1 GB of activations and gradients)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "executed_flops_per_step": flops,
        "step_frac_of_bf16_peak": dict(tensor_fracs(value / world, peaks), source=peaks["source"]),
        "full_backprop": {"ms_per_step": full_ms, "tflops": full_flops / (full_ms * 1e-3) / 1e12,
                          "frac": tensor_fracs(full_flops / (full_ms * 1e-3) / 1e12, peaks),
                          "executed_flops_per_step": full_flops, "elastic_speedup": full_ms / ms},
        "forward_ms": fwd_ms,
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": dY_host.numel() * dY_host.element_size(),
                "d2h_bytes_per_step": imp_host.numel() * 4},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "gemm_list_kernel (every GEMM of the step in one cooperative launch)", "bound": "tensor",
                     "achieved": ls_tf, "peak": peak, "unit": "TFLOP/s", "frac": ls_tf / peak,
                     "peak_source": peaks["source"] + (" cuBLAS bf16 burst" if use_burst else " cuBLAS bf16 sustained"),
                     "peak_choice": f"the timed region lasts {timed_span_s:.2f} s: " +
                                    ("burst peak (a kernel timed in a short run)" if use_burst else
                                     "sustained peak (a kernel timed inside a seconds-long step)"),
                     "frac_all": tensor_fracs(ls_tf, peaks),
                     "flops_per_launch": flops, "ms_per_launch": ls_ms, "launches_per_step": ls_n,
                     "ms_x_sm_mhz": (ls_ms * clocks["sm_mhz"]) if clocks.get("sm_mhz") else None,
                     "traffic": _list_traffic(args.blocks),
                     "traffic_note": "DRAM bytes per launch: ncu capture of the same launch on the 2-block stack "
                                     "(same shapes and token count), scaled by the GEMM flops of this stack"},
        "kernels": kernels,
    }
    if world == 1:
        # the oracle as it stands on the host cores: the sample the reference arm times, one warm-up call,
        # median of five
        times, fl, sample = time_oracle(w, 5, 1)
        line["cpu_baseline"] = {"value": fl / float(np.median(times)) / 1e12, "unit": UNIT, "cores": blas_threads(),
                                "kind": "oracle", "sample": sample, "seconds_per_step": float(np.median(times)),
                                "timed_steps": len(times), "warmup_steps": 1}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_selector(args):
    """Host-side selector report (Section 6.3): how many subproblems the two prunings remove, how the
    solution and the time of the dynamic program move with the resolution T_q (Eq. 8), and how the
    time falls with threads when there are thousands of tensors.  No GPU work."""
    import time
    import paper_2312_14227_b200 as et
    from workloads import flop_costs

    def timed(fn, reps=3):
        best = None
        for _ in range(reps):
            t0 = time.perf_counter()
            out = fn()
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        return out, 1e3 * best

    rng = np.random.default_rng(7)
    out = {"report": "selector (host dynamic program)"}
    # the ViT-L-shaped stack's 192 tensors with costs proportional to their work, rho = 0.5
    w = wl.vit_l(params=False)
    t_dw, t_dy = flop_costs(w.layers, w.M)
    I = rng.random(2 * w.L)
    t_fwd = 0.5 * float(t_dw.sum() + t_dy.sum()) / 2.0
    sweep = []
    ref_val = None
    for Tq in (10, 100, 1000, 10000, 100000):
        (mask, val, est, st), ms = timed(lambda: et.et_select_dp_ex(I, t_dw, t_dy, t_fwd, 0.5, Tq))
        (_, val_full, _, st_full), ms_full = timed(lambda: et.et_select_dp_ex(I, t_dw, t_dy, t_fwd, 0.5, Tq, prune=False), 1) \
            if Tq <= 10000 else ((None, val, None, None), None)
        assert abs(val_full - val) < 1e-9
        budget = 0.5 * (t_fwd + t_dw.sum() + t_dy.sum()) - t_fwd
        sweep.append({"Tq": Tq, "value": val, "selected": int(mask.sum()), "time_over_budget": float(est / budget),
                      "dp_ms": ms, "dp_ms_unpruned": ms_full, "subproblems_unpruned": st["table_full"],
                      "without_invalid": st["table_budget"], "visited": st["visited"],
                      "reduction": st["table_full"] / max(st["visited"], 1)})
        ref_val = val
    for e in sweep:
        e["value_vs_finest"] = e["value"] / ref_val
    out["vit_l_192_tensors_rho_0.5"] = sweep
    # thousands of tensors
    big = []
    for n, Tq in ((2048, 2000), (4096, 4000)):
        I2, w2, y2 = wl.selector_instance(rng, n, integer=False)
        row = {"n": n, "Tq": Tq, "rho": 0.4}
        base = None
        for threads in (1, 4, 16):
            (mask, val, est, st), ms = timed(lambda: et.et_select_dp_ex(I2, w2, y2, 10.0, 0.4, Tq, threads=threads), 2)
            base = val if base is None else base
            assert val == base
            row[f"ms_{threads}_threads"] = ms
            row["threads_used_%d" % threads] = st["threads"]
        row["transitions"] = st["transitions"]
        big.append(row)
    out["large_instances"] = big
    out["host_cores"] = os.cpu_count()
    print(json.dumps(out))


def run_dp_budget(args):
    """The ViT-B-shaped stack with masks from the host selector at time budgets rho of the full backward pass
    (per-tensor times measured on this GPU, seeded Uniform(0,1) importances, T_fwd = 0, T_q = 1000): per rho the
    selection, the time the model of Section 2.2 predicts for it and the measured step time."""
    import torch
    import paper_2312_14227_b200 as et

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    w = wl.vit_b() if args.blocks == 12 else wl.vit_b(n_blocks=args.blocks)
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(dev).contiguous()
    stack = et.et_stack_create(w.layers, w.M, w.dtype)
    W, b = [to_dev(a) for a in w.W], [to_dev(a) for a in w.b]
    ws = torch.empty(et.et_stack_workspace_bytes(stack), dtype=torch.uint8, device=dev)
    et.et_stack_bind(stack, W, b, ws)
    x, target = to_dev(w.x), to_dev(w.target)
    y = torch.empty((w.M, w.layers[-1].out_width), dtype=torch.bfloat16, device=dev)
    dY = torch.empty_like(y)
    et.et_forward_stack(stack, x, y)
    et.et_loss_mse_grad(stack, y, target, dY, None)
    t_dw, t_dy, t_fwd = et.et_profile_costs(stack, x, y, dY, iters=20)
    et.et_forward_stack(stack, x, y)
    delta = [to_dev(d) for d in wl.draw_delta(w, 5)]
    imp = torch.zeros(2 * w.L, dtype=torch.float32, device=dev)
    rep_ = et.Report(w.L)
    I = np.random.default_rng(9).random(2 * w.L)
    total = float(t_dw.sum() + t_dy.sum())

    def measure(mask, two_streams):
        et.et_stack_set_option(stack, et.ET_OPTION_TWO_STREAMS, 1 if two_streams else 0)
        for _ in range(max(args.warmup, 3)):
            et.et_backward_elastic(stack, dY, mask, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep_)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            et.et_backward_elastic(stack, dY, mask, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep_)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    rows = []
    for rho in (0.25, 0.5, 1.0):
        t0 = time.perf_counter()
        mask, val, est = et.et_select_dp(I, t_dw, t_dy, 0.0, rho, 1000, et.ET_COST_STRICT)
        dp_ms = 1e3 * (time.perf_counter() - t0)
        one = measure(mask, False)
        two = measure(mask, True)
        rows.append({"rho": rho, "selected_tensors": int(mask.sum()), "objective": val, "selector_ms": dp_ms,
                     "budget_ms": rho * total, "estimated_ms": est,
                     "measured_ms_one_stream": one, "measured_over_estimated_one_stream": one / est if est > 0 else None,
                     "measured_ms_two_streams": two, "measured_over_estimated_two_streams": two / est if est > 0 else None,
                     "executed_tflops_two_streams": rep_.flops_executed / two / 1e9})
    assert et.et_device_status(stack) == et.ET_OK
    print(json.dumps({"report": w.name + " selector masks at time budgets (T_fwd = 0, T_q = 1000)",
                      "profiled_full_backward_ms": total, "profiled_forward_ms": t_fwd, "budgets": rows,
                      "note": "estimated = sum of per-tensor times measured one kernel at a time (the model of "
                              "Section 2.2); one stream runs the same kernels back to back, two streams overlap the "
                              "weight gradients with the error-gradient chain"}))


def run_side(args):
    """Side reports for the other workload shapes (not the benchmark line): one JSON line each.
    resnet: ResNet-50 conv4_x 1x1 stack, elastic vs full step time (launch-bound GEMMs).
    schedule: ViT-L-shaped stack, the 200-iteration elastic schedule (10-step all-tensor window every
    50 steps, importances from the weight change over the window, selector at rho = 0.4 on
    measured per-tensor times) against 200 full-backprop iterations."""
    import torch
    import paper_2312_14227_b200 as et
    from paper_2312_14227_b200.elastic_loop import ElasticLoop

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    nb = {} if args.blocks == 12 else {"n_blocks": args.blocks}     # --blocks: a reduced stack of the same shapes (profiling)
    w = {"resnet": wl.resnet_1x1, "prenorm": lambda: wl.vit_b_prenorm(**nb), "full": lambda: wl.vit_b_full(**nb),
         "bottleneck": wl.resnet_bottleneck, "bottleneck_bn": lambda: wl.resnet_bottleneck(bn=True),
         "schedule": wl.vit_l, "schedule_full": wl.vit_l_full}[args.workload]()
    tdt = torch.bfloat16
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(tdt).to(dev).contiguous()
    stack = et.et_stack_create(w.layers, w.M, w.dtype)
    W, b = [to_dev(a) for a in w.W], [to_dev(a) for a in w.b]
    ws = torch.empty(et.et_stack_workspace_bytes(stack), dtype=torch.uint8, device=dev)
    et.et_stack_bind(stack, W, b, ws)
    x, target = to_dev(w.x), to_dev(w.target)
    y = torch.empty((w.M, w.layers[-1].out_width), dtype=tdt, device=dev)
    dY = torch.empty_like(y)
    et.et_forward_stack(stack, x, y)
    et.et_loss_mse_grad(stack, y, target, dY, None)
    torch.cuda.synchronize()
    if args.workload in ("resnet", "prenorm", "full", "bottleneck", "bottleneck_bn"):
        rep = et.Report(w.L)
        all_trainable = np.ones(2 * w.L, dtype=np.uint8)
        for l, ly in enumerate(w.layers):
            if ly.kind in (wl.KIND_ATTENTION, wl.KIND_IM2COL):   # a layer without tensors cannot be selected
                all_trainable[2 * l] = all_trainable[2 * l + 1] = 0
        delta = [to_dev(d) for d in wl.draw_delta(w, 5)]
        imp = torch.zeros(2 * w.L, dtype=torch.float32, device=dev)

        def timed(mask):
            for _ in range(5):
                et.et_backward_elastic(stack, dY, mask, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(args.steps):
                et.et_backward_elastic(stack, dY, mask, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps, rep.flops_executed, rep.launches

        ms, fl, n = timed(w.mask)
        fms, ffl, fn = timed(all_trainable)

        # the same elastic step replayed from a CUDA graph (the caller captures the library call)
        def graph_ms(mask):
            cap = torch.cuda.Stream()
            cap.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(cap):
                et.et_backward_elastic(stack, dY, mask, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep, stream=cap)
                cap.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=cap):
                    et.et_backward_elastic(stack, dY, mask, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep, stream=cap)
                for _ in range(5):
                    g.replay()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                cap.synchronize()
                e0.record(cap)
                for _ in range(args.steps):
                    g.replay()
                e1.record(cap)
                cap.synchronize()
            return e0.elapsed_time(e1) / args.steps

        try:
            gms, gfms = graph_ms(w.mask), graph_ms(all_trainable)
        except Exception as exc:                      # report, do not hide
            gms = gfms = None
            print("graph capture failed:", exc, file=sys.stderr)
        extra = {}
        if args.workload in ("bottleneck", "bottleneck_bn"):
            # the gather kernels alone: forward writes k*k times the activation, backward reads as much
            et.et_timing_enable(stack, True)
            for _ in range(5):
                et.et_forward_stack(stack, x, y)
                et.et_backward_elastic(stack, dY, all_trainable, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep)
            t = et.et_timing_read(stack)
            et.et_timing_enable(stack, False)
            g = [ly for ly in w.layers if ly.kind == wl.KIND_IM2COL]
            nbytes = sum(2.0 * (w.M * ly.in_features + w.M * ly.out_features) * 2 for ly in g)   # fwd + bwd, bf16
            gather_ms = t["attention"][0] / 5
            # no gather kernel runs where the GEMMs fetch the patches themselves (bf16, channels a multiple of 128)
            extra = {"gather_ms_per_forward_plus_backward": gather_ms, "gather_launches": t["attention"][1] / 5,
                     "gather_gbs": nbytes / gather_ms / 1e6 if gather_ms > 0 else None,
                     "gather_frac_of_hbm_peak": nbytes / gather_ms / 1e6 / _peaks()["hbm_gbs"] if gather_ms > 0 else None,
                     "dgrad_ms": t["dgrad"][0] / 5, "wgrad_ms": t["wgrad"][0] / 5, "forward_gemm_ms": t["forward"][0] / 5,
                     "norm_ms_per_forward_plus_backward": t["norm"][0] / 5, "norm_timed_regions": t["norm"][1] / 5}
        if args.workload == "full":
            # the attention kernels alone, over full-backprop steps: 4 S^2 64 flops per (sequence, head)
            # forward, 2.5 times that backward (five GEMMs, one of them the recomputed scores)
            ones = all_trainable
            et.et_timing_enable(stack, True)
            for _ in range(5):
                et.et_forward_stack(stack, x, y)
                et.et_backward_elastic(stack, dY, ones, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep)
            t = et.et_timing_read(stack)
            et.et_timing_enable(stack, False)
            att = [ly for ly in w.layers if ly.kind == wl.KIND_ATTENTION]
            fwd_flops = sum(4.0 * (w.M // ly.seq) * ly.heads * ly.seq * ly.seq * 64 for ly in att)
            att_ms = t["attention"][0] / 5
            extra = {"attention_ms_per_forward_plus_backward": att_ms, "attention_launches": t["attention"][1] / 5,
                     "attention_tflops": 3.5 * fwd_flops / att_ms / 1e9, "norm_ms": t["norm"][0] / 5,
                     "dgrad_ms": t["dgrad"][0] / 5, "wgrad_ms": t["wgrad"][0] / 5, "forward_gemm_ms": t["forward"][0] / 5}
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(args.steps):
                et.et_forward_stack(stack, x, y)
            e1.record()
            torch.cuda.synchronize()
            extra["forward_ms"] = e0.elapsed_time(e1) / args.steps
        if args.workload == "prenorm":
            # normalisation kernels alone: CUDA-event time of their class over full-backprop steps against
            # the bytes they must move (g, x, skip gradient in; error gradient out; bf16)
            ones = np.ones(2 * w.L, dtype=np.uint8)
            et.et_timing_enable(stack, True)
            for _ in range(5):
                et.et_backward_elastic(stack, dY, ones, None, delta, imp, et.ET_FLAG_FUSE_SGD, w.lr, rep)
            t = et.et_timing_read(stack)
            et.et_timing_enable(stack, False)
            n_norm = sum(1 for l, ly in enumerate(w.layers) if ly.kind == wl.KIND_NORM and l > 0)
            nbytes = n_norm * 4.0 * w.M * w.layers[0].out_features * 2
            norm_ms = t["norm"][0] / 5
            peaks = _peaks()
            extra = {"norm_backward_ms_per_step": norm_ms, "norm_launches_per_step": t["norm"][1] / 5,
                     "norm_backward_gbs": nbytes / norm_ms / 1e6,
                     "norm_frac_of_hbm_peak": nbytes / norm_ms / 1e6 / peaks["hbm_gbs"],
                     "norm_note": "class time includes the gamma finishing kernels; bytes count the row kernels only"}
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(args.steps):
                et.et_forward_stack(stack, x, y)
            e1.record()
            torch.cuda.synchronize()
            extra["forward_ms"] = e0.elapsed_time(e1) / args.steps
        print(json.dumps({"report": w.name, **extra, "elastic_ms": ms, "elastic_tflops": fl / ms / 1e9,
                          "elastic_launches": n, "full_ms": fms, "full_tflops": ffl / fms / 1e9, "full_launches": fn,
                          "elastic_graph_ms": gms, "full_graph_ms": gfms,
                          "selected_tensors": int(w.mask.sum())}))
        return
    t_dw, t_dy, t_fwd = et.et_profile_costs(stack, x, y, dY, iters=10)
    loop = ElasticLoop(stack, W, b, x, target, w.lr, 50, 10, 0.4, t_dw, t_dy, t_fwd=t_fwd, Tq=1000, master=True)
    W0, b0 = [t.clone() for t in W], [t.clone() for t in b]

    def restore():
        for dst, src in zip(W + b, W0 + b0):
            dst.copy_(src)
        for dst, src in zip(loop.W32 + loop.b32, W0 + b0):
            dst.copy_(src)

    loop.run(10, elastic=False)                                   # warm-up
    restore()
    full = loop.run(200, elastic=False, time_steps=True)
    restore()
    el = loop.run(200, elastic=True, time_steps=True)
    T_full = t_fwd + t_dw.sum() + t_dy.sum()
    est = [t_fwd + et.et_time_selective(m, t_dw, t_dy) for m in el["masks"]]
    print(json.dumps({"report": w.name + " elastic schedule, 200 iterations", "rho": 0.4,
                      "full_ms_per_step": full["ms_per_step"], "elastic_ms_per_step": el["ms_per_step"],
                      "ratio": el["ms_per_step"] / full["ms_per_step"],
                      "model_estimate_ratio": float(np.mean(est) / T_full),
                      "selected_tensors_per_period": [int(m.sum()) for m in el["masks"][10::50]],
                      "selector_ms": el["dp_ms"], "profiled_full_step_ms": float(T_full),
                      "loss_first_last": [float(el["losses"][0]), float(el["losses"][-1])],
                      "note": "includes forward, loss, host selector and snapshot copies; bf16 storage "
                              "with fp32 master weights"}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--blocks", type=int, default=12, help="transformer blocks of the stack (12 = the benchmark workload)")
    ap.add_argument("--profile", action="store_true",
                    help="short run for ncu: one forward and two all-selected backward steps, no timing")
    ap.add_argument("--plain-launch", action="store_true",
                    help="launch the one-launch backward as a plain (not cooperative) grid: for runs under a profiler, "
                         "which does not take the cooperative launch")
    ap.add_argument("--optimizer", default="sgd", choices=["sgd", "sgdw", "adam"],
                    help="update fused into the step: plain SGD (the benchmark line) or the paper's SGDW / Adam")
    ap.add_argument("--workload", default="vit_b", choices=["vit_b", "dp_budget", "resnet", "prenorm", "full", "bottleneck", "bottleneck_bn", "schedule", "schedule_full", "selector"],
                    help="vit_b = the benchmark line; resnet / prenorm / schedule = side reports for the other shapes; "
                         "selector = host-side report on the selection dynamic program")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "own" else args.warmup
    if args.workload == "selector":
        run_selector(args)
    elif args.workload == "dp_budget":
        run_dp_budget(args)
    elif args.workload != "vit_b":
        run_side(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_own(args)


if __name__ == "__main__":
    main()
