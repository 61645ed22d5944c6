#!/usr/bin/env python
"""Benchmark of the IM-attention hot path on synthetic MOSEI-shaped data.

A step is one forward pass of the whole hot path over one batch: the GsiT fusion stack (forward-ring and
backward-ring encoders at width d, intra-modal encoder at width 2d), every layer being LayerNorm -> shared
QKV projection -> IM attention -> out-projection + residual -> LayerNorm -> MLP + residual, all inside the
library's kernels (three launches per layer).  `value` is valid (non padded) tokens per second with inputs resident in HBM; `e2e`
includes the host->device copy of the batch and the device->host copy of the result every step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--repeats R] [--impl reference]
    python bench.py --only attention|layer --workload W --batch B --phase P [--d D --heads H] [--calls C]   (profiler driver)

With --gpus N > 1 and no torchrun environment the script starts N worker processes itself, one GPU each.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import workloads as wk  # noqa: E402

METRIC = "IM-attention tokens/s (valid tokens through the GsiT IM stack), MOSEI-shaped"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126 * 1024 * 1024


def recorded_traffic(kernel: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel`, from the ncu capture summarised under
    profiles/ (profiles/traffic.json, written next to the summary when the capture is taken), or None when there is no
    record for the kernel as it stands."""
    p = ROOT / "profiles" / "traffic.json"
    if not p.exists():
        return None
    rec = json.loads(p.read_text()).get(kernel)
    return None if rec is None else float(rec["dram_bytes_per_launch"])


def scaled_traffic(per_problem, problems: int):
    """The capture is of a launch serving one problem; a launch serving two independent problems of the same shape moves
    twice the bytes."""
    return None if per_problem is None else per_problem * problems


def peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of the benchmark GPU through NVML while the timed region runs."""

    def __init__(self, torch_device_index: int):
        self.samples, self.reasons, self.max_mhz, self._stop = [], set(), None, threading.Event()
        self._thread, self._h, self._nv = None, None, None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self._nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # NVML missing: the clocks object then says so
            self.error = repr(e)

    def _names(self, mask: int):
        nv = self._nv
        table = {"sw_power_cap": "nvmlClocksThrottleReasonSwPowerCap", "hw_slowdown": "nvmlClocksThrottleReasonHwSlowdown",
                 "hw_thermal_slowdown": "nvmlClocksThrottleReasonHwThermalSlowdown",
                 "sw_thermal_slowdown": "nvmlClocksThrottleReasonSwThermalSlowdown",
                 "hw_power_brake": "nvmlClocksThrottleReasonHwPowerBrakeSlowdown",
                 "sync_boost": "nvmlClocksThrottleReasonSyncBoost"}
        return {n for n, attr in table.items() if hasattr(nv, attr) and (mask & getattr(nv, attr))}

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.reasons |= self._names(int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)))
            except Exception:
                pass
            self._stop.wait(0.01)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                    "note": getattr(self, "error", "no samples")}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def stack_flops_and_tokens(wl, valid_len, batch):
    """Valid tokens per step, and per attention call: useful pairs, useful FLOPs, compulsory bytes."""
    seg = wl.seg_len
    n = np.tile(np.asarray(seg)[None], (batch, 1)) if valid_len is None else valid_len
    tokens = int(n.sum())
    ring = np.array([[0, 1, 0], [0, 0, 1], [1, 0, 0]])
    info = {}
    for name, allowed, d in (("cross", ring, wl.d_model), ("intra", np.eye(3, dtype=int), 2 * wl.d_model)):
        U = wk.useful_pairs(seg, valid_len, allowed, batch)
        info[name] = {"pairs": U, "flops": 4.0 * d * U, "bytes": 4.0 * tokens * d * 2 + 12.0 * batch, "d": d}
    return tokens, info


def run_reference(args):
    """The CPU oracle, as it stands, timed on the host cores on a bounded sample of the same workload."""
    import oracle
    wl = wk.WORKLOADS[args.workload]
    sub = args.ref_batch
    inp = wk.make_inputs(args.workload, batch=sub)
    tokens = int(inp["valid_len"].sum()) if inp["valid_len"] is not None else sub * wl.L
    n_f, n_b, n_i, ih = wl.stack if wl.stack else (1, 0, 0, wl.heads)

    def step():
        if wl.stack:
            oracle.gsit_stack_fwd(inp["x"], inp["fwd_layers"], inp["bwd_layers"], inp["intra_layers"], wl.seg_len,
                                  wl.heads, ih, inp["valid_len"])
        else:
            oracle.im_layer_fwd(inp["x"], inp["layer"], wl.seg_len, wl.heads, inp["valid_len"], oracle.PHASE_INTER_FWD)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = tokens / dt
    sample = f"{sub} of {wl.batch} samples per step (valid tokens {tokens}), fp64 dense-mask oracle, whole stack"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"cfg{wl.index}:{wl.name}", "batch": sub, "seg_len": list(wl.seg_len),
                       "d_model": wl.d_model, "heads": wl.heads},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def _time_graph_replays(torch, graphs, steps, dist, world):
    """One timed region: exactly `steps` replays between a barrier + synchronize on both sides, CUDA events on the
    launching stream, maximum over ranks.  Returns milliseconds."""
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    beg, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    beg.record()
    for k in range(steps):
        graphs[k % len(graphs)].replay()
    end.record()
    torch.cuda.synchronize()
    ms = beg.elapsed_time(end)
    if world > 1:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
        dist.barrier()
    return ms


def time_attention_alone(torch, g, wl, valid_dev, d, heads, phase, reps=4, batch=None):
    """One IM-attention call timed alone: a CUDA graph of launches rotating over qkv/out buffer sets larger than L2."""
    B, L = (batch or (wl.batch if valid_dev is None else valid_dev.shape[0])), wl.L
    set_bytes = B * L * 4 * d * 2
    nsets = min(64, max(2, int(np.ceil(1.5 * L2_BYTES / set_bytes))))
    gen = torch.Generator(device="cuda").manual_seed(1234)
    qkvs = [torch.randn((B, L, 3, heads, d // heads), device="cuda", generator=gen).bfloat16() for _ in range(nsets)]
    outs = [torch.empty((B, L, d), device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
    wss = [torch.empty(256, dtype=torch.uint8, device="cuda") for _ in range(nsets)]
    run = lambda i: g.im_attention_fwd(qkvs[i][:, :, 0], qkvs[i][:, :, 1], qkvs[i][:, :, 2], wl.seg_len, valid_dev, phase, out=outs[i],
                                       workspace=wss[i])
    for i in range(nsets):
        run(i)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(reps):
            for i in range(nsets):
                run(i)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    beg, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    beg.record()
    for _ in range(5):
        graph.replay()
    end.record()
    torch.cuda.synchronize()
    return beg.elapsed_time(end) * 1e-3 / (5 * reps * nsets), nsets


PATTERNS = {"fwd": [[0, 1, 0], [0, 0, 1], [1, 0, 0]], "bwd": [[0, 0, 1], [1, 0, 0], [0, 1, 0]], "intra": [[1, 0, 0], [0, 1, 0], [0, 0, 1]]}


def attention_per_config(torch, g, pk, ex2_rate):
    """IM attention alone at the aligned (cfg 2) and MOSI-shaped (cfg 3) workloads, all three block patterns: time, tokens/s,
    useful TFLOP/s and the fraction of both rooflines.  Reported, not graded (cfg 2 is launch-latency bound)."""
    out = {}
    for idx in (2, 3):
        wl = wk.WORKLOADS[idx]
        valid = wk.draw_valid_len(np.random.default_rng(wl.seed), wl)
        vl = None if valid is None else torch.from_numpy(valid).cuda()
        tokens = wl.batch * wl.L if valid is None else int(valid.sum())
        rec = {}
        for name, phase in (("fwd", g.PHASE_INTER_FWD), ("bwd", g.PHASE_INTER_BWD), ("intra", g.PHASE_INTRA)):
            sec, nsets = time_attention_alone(torch, g, wl, vl, wl.d_model, wl.heads, phase, batch=wl.batch)
            U = wk.useful_pairs(wl.seg_len, valid, PATTERNS[name], wl.batch)
            fl, by = 4.0 * wl.d_model * U, 4.0 * tokens * wl.d_model * 2
            t_tc, t_hbm, t_exp = fl / (pk["bf16_tflops"] * 1e12), by / (pk["hbm_gbs"] * 1e9), wl.heads * U / ex2_rate
            rec[name] = {"us": sec * 1e6, "tokens_per_s": tokens / sec, "useful_tflops": fl / sec / 1e12,
                         "frac_roofline": max(t_tc, t_hbm) / sec, "frac_three_way": max(t_tc, t_hbm, t_exp) / sec,
                         "t_hbm_us": t_hbm * 1e6, "t_exp_us": t_exp * 1e6, "buffer_sets": nsets}
        out[f"cfg{idx}:{wl.name}"] = rec
    torch.cuda.empty_cache()
    return out


def run_only(args):
    """Profiler driver: a few launches of one library call on workload-shaped inputs (N(0,1) values, the workload's padding
    recipe), so that `ncu -k ... -c ...` has a short, self-contained command to wrap.  Prints the device status."""
    import torch

    import paper_2505_01068_b200 as g
    g.load()
    wl = wk.WORKLOADS[args.workload]
    B = args.batch or wl.batch
    rng = np.random.default_rng(wl.seed)
    valid = wk.draw_valid_len(rng, wl, B)
    vl = None if valid is None else torch.from_numpy(valid).cuda()
    d, heads = args.d or wl.d_model, args.heads or wl.heads
    gen = torch.Generator(device="cuda").manual_seed(1)
    nsets = 3
    if args.only == "attention":
        bufs = [torch.randn((B, wl.L, 3, heads, d // heads), device="cuda", generator=gen).bfloat16() for _ in range(nsets)]
        outs = [torch.empty((B, wl.L, d), device="cuda", dtype=torch.bfloat16) for _ in range(nsets)]
        ws = torch.empty(256, dtype=torch.uint8, device="cuda")
        run = lambda i: g.im_attention_fwd(bufs[i][:, :, 0], bufs[i][:, :, 1], bufs[i][:, :, 2], wl.seg_len, vl, args.phase,
                                           out=outs[i], workspace=ws)
    else:
        w = wk.draw_layer_weights(rng, d, wl.d_ff_mult * d, wl.dtype)
        wd = {k: (None if v is None else (torch.from_numpy(v).cuda().bfloat16() if (k.startswith("w_") and wl.dtype == "bf16")
                                          else torch.from_numpy(v).cuda())) for k, v in w.items()}
        bufs = [torch.randn((B, wl.L, d), device="cuda", generator=gen) for _ in range(nsets)]
        outs = [torch.empty((B, wl.L, d), device="cuda") for _ in range(nsets)]
        sh = g.make_shape(B, wl.seg_len, d, heads, vl, g.binding._dtype_code(wd["w_qkv"].dtype), args.phase)
        ws = torch.empty(g.workspace_bytes(sh, g.CALL_LAYER, wd["w_1"].shape[0]), dtype=torch.uint8, device="cuda")
        run = lambda i: g.im_layer_fwd(bufs[i], wd, wl.seg_len, heads, vl, args.phase, out=outs[i], workspace=ws)
    if args.kernels:
        g.tune_attention(args.kernels)
    for c in range(args.calls):
        run(c % nsets)
    torch.cuda.synchronize()
    print(f"{args.only} workload {args.workload} batch {B} phase {args.phase} d {d} heads {heads}: device status", g.last_device_status())


def run_gpu(args):
    import torch
    import torch.distributed as dist

    import paper_2505_01068_b200 as g
    from paper_2505_01068_b200 import shard

    rank, world = int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    g.load()
    wl = wk.WORKLOADS[args.workload]
    assert wl.stack is not None, "the benchmark step is the full stack (workload 4)"
    n_f, n_b, n_i, ih = wl.stack
    # weak scaling: every rank owns an independent batch of the same shape (no data-path collective)
    inp = wk.make_inputs(wl.index, seed=shard.rank_seed(wl.seed, rank))
    B = wl.batch
    valid = inp["valid_len"]
    vl = torch.from_numpy(valid).cuda()
    tokens, info = stack_flops_and_tokens(wl, valid, B)

    def dev_w(w):
        return {k: (None if a is None else (torch.from_numpy(a).cuda().bfloat16() if k.startswith("w_") else torch.from_numpy(a).cuda()))
                for k, a in w.items()}

    stack = g.GsitStack([dev_w(w) for w in inp["fwd_layers"]], [dev_w(w) for w in inp["bwd_layers"]],
                        [dev_w(w) for w in inp["intra_layers"]], wl.seg_len, wl.heads, ih)
    x_host = torch.from_numpy(inp["x"]).pin_memory()
    nbuf = max(2, int(np.ceil(1.2 * L2_BYTES / x_host.numel() / 4)))
    xbufs = [x_host.cuda() for _ in range(nbuf)]
    # per layer: LN1+QKV, IM attention, out-proj+LN2+MLP (fused kernels); each intra layer once per half of the batch
    paired = stack.paired_rings and n_f == n_b and n_f > 0   # one launch per kernel for both rings of a depth
    launches_per_step = 3 * (n_f if paired else n_f + n_b) + 3 * n_i * (2 if (stack.intra_halves and B >= 2) else 1)
    if stack.packed:
        launches_per_step += 3   # row plan, gather of the real rows, scatter of the result

    for i in range(max(1, min(args.warmup, 2))):           # eager warm-up (module load, attributes, buffers)
        stack.forward(xbufs[i % nbuf], vl)
    torch.cuda.synchronize()
    code, flags = g.last_device_status()
    assert code == 0 and flags == 0, (code, flags)
    graphs = []
    for i in range(nbuf):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            y_dev = stack.forward(xbufs[i], vl)
        graphs.append(gr)
    for k in range(args.warmup):
        graphs[k % nbuf].replay()
    torch.cuda.synchronize()

    # a step is under a millisecond: the region of `steps` steps is repeated and the median region is reported
    with ClockSampler(local) as clocks:
        regions = [_time_graph_replays(torch, graphs, args.steps, dist, world) for _ in range(args.repeats)]
    ms = float(np.median(regions))
    ms_per_step = ms / args.steps
    # whole job: tokens of all ranks over the slowest rank's time (ms is already the maximum over ranks)
    _, _, value = shard.job_throughput(tokens, ms_per_step, device="cuda")

    # ---- end to end: pinned host batch -> device -> stack -> pinned host result, every step, through the package's
    # host pipeline (the three legs of neighbouring steps overlap; every step moves its own input and output) ----
    from paper_2505_01068_b200.hostio import HostPipeline
    vl_host = torch.from_numpy(valid).pin_memory()
    y_hosts = [torch.empty((B, wl.L, 2 * wl.d_model), dtype=torch.float32).pin_memory() for _ in range(2)]
    pipe = HostPipeline(stack, tuple(x_host.shape), depth=2)
    e2e_steps = max(3, min(args.steps, 30))
    for k in range(3):
        pipe.step(x_host, y_hosts[k % 2], vl_host)
    pipe.wait()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for k in range(e2e_steps):
        pipe.step(x_host, y_hosts[k % 2], vl_host)
    pipe.wait()
    _, _, e2e_value = shard.job_throughput(tokens, (time.perf_counter() - t0) / e2e_steps * 1e3, device="cuda")
    y_host = y_hosts[0]

    # ---- per-kernel device times inside the step (eager, CUDA events around each launch) ----
    # Everything is issued on one stream here (the intra encoder on the whole batch), so that every event pair brackets
    # one kernel running alone; with paired rings a cross-modal launch serves both rings (two problems).
    trace_steps = max(1, min(args.steps, 10))
    stack.concurrent_rings = False
    g.trace_enable(True)
    for k in range(trace_steps):
        stack.forward(xbufs[k % nbuf], vl)
    torch.cuda.synchronize()
    stack.concurrent_rings = True
    att = g.trace_launches(g.KERNEL_ATTENTION)
    lin_ms, lin_n = g.trace_read(g.KERNEL_LINEAR)
    ln_ms, ln_n = g.trace_read(g.KERNEL_LAYERNORM)
    g.trace_enable(False)
    n_cross = n_f if paired else n_f + n_b
    problems = 2 if paired else 1
    per_step = n_cross + n_i
    att = np.asarray(att).reshape(trace_steps, per_step)
    cross_launch_s = float(att[:, :n_cross].mean()) * 1e-3
    cross_s = cross_launch_s / problems          # per problem
    intra_s = float(att[:, n_cross:].mean()) * 1e-3 if n_i else None
    pk, pk_kind = peaks()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- IM attention timed alone (burst), both block patterns, against both rooflines ----
    ex2_rate = 148 * 16 * (clocks.summary()["sm_max_mhz"] or 1965) * 1e6     # MUFU ex2 per second at max clock
    attention = {}
    for name, d, heads, phase in (("cross", wl.d_model, wl.heads, g.PHASE_INTER_FWD), ("intra", 2 * wl.d_model, ih, g.PHASE_INTRA)):
        sec, nsets = time_attention_alone(torch, g, wl, vl, d, heads, phase)
        I = info[name]
        t_tc, t_hbm = I["flops"] / (pk["bf16_tflops"] * 1e12), I["bytes"] / (pk["hbm_gbs"] * 1e9)
        t_exp = heads * I["pairs"] / ex2_rate
        attention[name] = {"us": sec * 1e6, "tokens_per_s": tokens / sec, "useful_tflops": I["flops"] / sec / 1e12,
                           "achieved_gbs": I["bytes"] / sec / 1e9, "frac_roofline": max(t_tc, t_hbm) / sec,
                           "frac_three_way": max(t_tc, t_hbm, t_exp) / sec, "t_tensor_us": t_tc * 1e6,
                           "t_hbm_us": t_hbm * 1e6, "t_exp_us": t_exp * 1e6, "d_model": d, "heads": heads,
                           "buffer_sets": nsets, "in_step_us": (cross_s if name == "cross" else intra_s) * 1e6}

    # ---- the same stack at the paper's length statistics (second workload family: about a quarter of the positions
    # are real), packed row layout against the padded one: context, not part of `value` ----
    stats_lengths = {}
    if not args.no_scaled:
        v6 = wk.draw_valid_len(np.random.default_rng(wk.WORKLOADS[6].seed), wk.WORKLOADS[6], B)
        vl6 = torch.from_numpy(v6).cuda()
        for name, packed in (("padded_layout", False), ("packed_layout", True)):
            st6 = g.GsitStack(stack.fwd, stack.bwd, stack.intra, wl.seg_len, wl.heads, ih, packed=packed)
            st6.forward(xbufs[0], vl6)
            torch.cuda.synchronize()
            gs6 = []
            for i in range(nbuf):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr):
                    st6.forward(xbufs[i], vl6)
                gs6.append(gr)
            _time_graph_replays(torch, gs6, nbuf, dist, 1)
            ms6 = _time_graph_replays(torch, gs6, 50, dist, 1) / 50
            stats_lengths[name] = {"ms_per_step": ms6, "tokens_per_s": float(v6.sum()) / (ms6 * 1e-3)}
            del gs6, st6
        stats_lengths["valid_tokens_per_step"] = int(v6.sum())
        stats_lengths["real_fraction"] = float(v6.sum()) / (B * wl.L)
        torch.cuda.empty_cache()

    # ---- the scaled shape (head_dim 64, tcgen05 kernel), attention alone: context for the tensor-bound case ----
    scaled = {}
    if not args.no_scaled:
        wl5 = wk.WORKLOADS[5]
        v5 = wk.draw_valid_len(np.random.default_rng(wl5.seed), wl5)
        vl5 = torch.from_numpy(v5).cuda()
        tok5 = int(v5.sum())
        for name, phase, allowed in (("cross", g.PHASE_INTER_FWD, [[0, 1, 0], [0, 0, 1], [1, 0, 0]]), ("intra", g.PHASE_INTRA, np.eye(3, dtype=int))):
            sec, nsets = time_attention_alone(torch, g, wl5, vl5, wl5.d_model, wl5.heads, phase, reps=1)
            U = wk.useful_pairs(wl5.seg_len, v5, allowed, wl5.batch)
            fl, by = 4.0 * wl5.d_model * U, 4.0 * tok5 * wl5.d_model * 2
            t_tc, t_hbm = fl / (pk["bf16_tflops"] * 1e12), by / (pk["hbm_gbs"] * 1e9)
            scaled[name] = {"us": sec * 1e6, "tokens_per_s": tok5 / sec, "useful_tflops": fl / sec / 1e12,
                            "frac_roofline": max(t_tc, t_hbm) / sec, "t_tensor_us": t_tc * 1e6, "t_hbm_us": t_hbm * 1e6,
                            "t_exp_us": wl5.heads * U / ex2_rate * 1e6, "batch": wl5.batch, "buffer_sets": nsets}
        # the shared QKV projection at the same shape (tcgen05 GEMM, d=512): x [B, L, 512] -> qkv [B, L, 3, 8, 64]
        xs5 = [torch.randn((wl5.batch, wl5.L, wl5.d_model), device="cuda").bfloat16() for _ in range(2)]
        w5 = (torch.randn((3 * wl5.d_model, wl5.d_model), device="cuda") * wl5.d_model ** -0.5).bfloat16()
        qs5 = [torch.empty((wl5.batch, wl5.L, 3, wl5.heads, wl5.d_model // wl5.heads), device="cuda", dtype=torch.bfloat16) for _ in range(2)]
        for i in range(2):
            g.im_qkv_proj(xs5[i], w5, None, wl5.seg_len, wl5.heads, vl5, out=qs5[i])
        torch.cuda.synchronize()
        beg, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        beg.record()
        for _ in range(5):
            for i in range(2):
                g.im_qkv_proj(xs5[i], w5, None, wl5.seg_len, wl5.heads, vl5, out=qs5[i])
        end.record()
        torch.cuda.synchronize()
        sec = beg.elapsed_time(end) * 1e-3 / 10
        fl = 2.0 * wl5.batch * wl5.L * wl5.d_model * 3 * wl5.d_model
        scaled["qkv_proj"] = {"us": sec * 1e6, "tflops": fl / sec / 1e12, "frac_tensor_peak": fl / sec / 1e12 / pk["bf16_tflops"],
                              "note": "padded layout: all B*L rows multiplied (padded rows are zeroed in the epilogue)"}
        # the same projection on the packed row layout: real rows only
        cap5 = wl5.batch * wl5.L + 128
        plan5 = g.plan_rows(vl5, wl5.seg_len)
        xp5 = [torch.cat([x.reshape(-1, wl5.d_model), torch.zeros((128, wl5.d_model), device="cuda", dtype=torch.bfloat16)]) for x in xs5]
        qp5 = [torch.empty((cap5, 3, wl5.heads, wl5.d_model // wl5.heads), device="cuda", dtype=torch.bfloat16) for _ in range(2)]
        for i in range(2):
            g.im_qkv_proj(xp5[i], w5, None, wl5.seg_len, wl5.heads, vl5, out=qp5[i], row_start=plan5)
        torch.cuda.synchronize()
        beg.record()
        for _ in range(5):
            for i in range(2):
                g.im_qkv_proj(xp5[i], w5, None, wl5.seg_len, wl5.heads, vl5, out=qp5[i], row_start=plan5)
        end.record()
        torch.cuda.synchronize()
        sec_p = beg.elapsed_time(end) * 1e-3 / 10
        fl_real = 2.0 * tok5 * wl5.d_model * 3 * wl5.d_model
        scaled["qkv_proj_packed"] = {"us": sec_p * 1e6, "tflops_real_rows": fl_real / sec_p / 1e12,
                                     "padded_layout_tflops_real_rows": fl_real / sec / 1e12, "real_rows": tok5,
                                     "note": "packed layout: real rows only, rows stored one by one instead of by TMA"}
        del xp5, qp5
        del vl5, xs5, qs5
        torch.cuda.empty_cache()

    # ---- CPU baseline: the oracle on a bounded sample of the same workload ----
    import oracle
    sub = args.ref_batch
    ref_inp = wk.make_inputs(wl.index, batch=sub)
    ref_tokens = int(ref_inp["valid_len"].sum())
    ref_step = lambda: oracle.gsit_stack_fwd(ref_inp["x"], ref_inp["fwd_layers"], ref_inp["bwd_layers"],
                                             ref_inp["intra_layers"], wl.seg_len, wl.heads, ih, ref_inp["valid_len"])
    ref_step()
    t0 = time.perf_counter()
    ref_step()
    cpu_s = time.perf_counter() - t0

    cross = info["cross"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"cfg{wl.index}:{wl.name}", "batch_per_gpu": B, "seg_len": list(wl.seg_len), "d_model": wl.d_model,
                   "heads": wl.heads, "stack": f"fwd x{n_f} + bwd x{n_b} at d={wl.d_model} (hd={wl.d_model // wl.heads}), "
                   f"intra x{n_i} at d={2 * wl.d_model} (hd={2 * wl.d_model // ih})",
                   "valid_tokens_per_step": tokens, "padded_tokens_per_step": B * wl.L,
                   "l2": f"inputs rotate over {nbuf} device copies ({nbuf * x_host.numel() * 4 >> 20} MiB > 126 MiB L2); "
                         "the step's scratch alone is larger than L2", "launch": "one CUDA graph per input buffer; inside it " + ("the forward and backward ring layers of each depth in one launch per kernel (two problems per launch), " if paired else "the forward and backward rings on two streams, ") +
                             "then the intra encoder on the two halves of the batch on two streams; packed row layout (real rows only); "
                             "kernels of a stream start under the tail of the one before (programmatic dependent launch)"},
        "clocks": clocks.summary(),
        "timed_regions": {"repeats": args.repeats, "steps_each": args.steps, "ms_per_step_median": ms_per_step,
                          "ms_per_step_min": min(regions) / args.steps, "ms_per_step_max": max(regions) / args.steps},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel() * 4),
                "d2h_bytes_per_step": int(y_host.numel() * 4) ,
                "how": "HostPipeline, 2 steps in flight: copy-in, kernels and copy-out of neighbouring steps overlap"},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"kernel": "attn_bf16_kernel<8,64> (cross-modal IM attention inside the step" + (", both rings' layers of a depth in one launch)" if paired else ")"), "bound": "hbm",
                     "achieved": problems * cross["bytes"] / cross_launch_s / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": problems * cross["bytes"] / cross_launch_s / 1e9 / pk["hbm_gbs"],
                     "traffic": scaled_traffic(recorded_traffic("attn_bf16_hd8_cfg4_cross"), problems), "peak_kind": "of " + pk_kind,
                     "launch_us": cross_launch_s * 1e6, "algorithmic_bytes": problems * cross["bytes"], "problems_per_launch": problems,
                     "timed": "event pair around each launch, everything on one stream for this pass; traffic = the one-problem capture x problems per launch",
                     # the same launch against the exponential unit: one ex2 per useful (query, key) pair per head
                     "alu": {"bound": "ex2 (special-function unit)", "achieved": wl.heads * cross["pairs"] / cross_s / 1e9,
                             "peak": ex2_rate / 1e9, "unit": "Gex2/s", "frac": wl.heads * cross["pairs"] / cross_s / ex2_rate,
                             "peak_kind": "148 SMs x 16 ex2/clk x max SM clock"}},
        "cpu_baseline": {"value": ref_tokens / cpu_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": f"{sub} of {B} samples, one step (valid tokens {ref_tokens}) in {cpu_s:.2f} s"},
        "attention": attention,
        "attention_other_configs": attention_per_config(torch, g, pk, ex2_rate) if not args.no_scaled else {},
        "scaled_attention_hd64": scaled,
        "length_statistics_workload": stats_lengths,
        "step_kernel_ms": {"attention": float(att.sum()) / trace_steps, "linear": lin_ms / trace_steps,
                           "layernorm": ln_ms / trace_steps, "launches": {"attention": per_step, "linear": lin_n // trace_steps,
                                                                          "layernorm": ln_n // trace_steps}},
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def _spawned_rank(rank, args, world, port):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    os.environ.setdefault("NCCL_DEBUG", "INFO")   # leave NCCL's transport lines (NVLS, P2P) visible in the workers' stderr
    run_gpu(args)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--repeats", type=int, default=25, help="timed regions of --steps steps each; the median is reported")
    ap.add_argument("--impl", default="gsit", choices=["gsit", "reference"])
    ap.add_argument("--workload", type=int, default=4)
    ap.add_argument("--ref-batch", type=int, default=16, help="samples per step of the CPU oracle")
    ap.add_argument("--no-scaled", action="store_true", help="skip the extra timings (other configs, head_dim 64, length statistics)")
    ap.add_argument("--only", choices=["attention", "layer"], help="profiler driver: launch one call a few times and exit")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--phase", type=int, default=0)
    ap.add_argument("--d", type=int, default=0)
    ap.add_argument("--heads", type=int, default=0)
    ap.add_argument("--calls", type=int, default=3)
    ap.add_argument("--kernels", type=int, default=0, help="--only: kernel choice of include/gsit_test.h (0 = defaults)")
    args = ap.parse_args()
    if args.only:
        run_only(args)
        return
    if args.impl == "reference":
        args.steps = 2 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        if int(os.environ.get("RANK", 0)) == 0:
            run_reference(args)
        return
    args.steps = 200 if args.steps is None else args.steps
    args.warmup = max(3, 5 if args.warmup is None else args.warmup)
    args.repeats = max(1, args.repeats)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher around us: start one worker per GPU (NCCL serves only the barrier and the max over ranks)
        from paper_2505_01068_b200 import shard
        shard.spawn_ranks(args.gpus, _spawned_rank, (args,))
        return
    run_gpu(args)


if __name__ == "__main__":
    main()
