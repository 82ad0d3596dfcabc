#!/usr/bin/env python
"""Benchmark of the activation-masked gated-MLP path on B200.

One "step" is one denoising step of the pi0-style action expert (18 layers, H=1024, I=4096, T=51, top-25 % masks
reused across steps): `rm_action_expert_step` with the device-resident index lists, plus -- once every 10 steps,
which is how often the workload derives its masks -- `rm_mask_compact` (top-k over the resident reference
records).  Inputs are resident in HBM for `value`; `e2e` goes through `rm_action_expert_step_host` with pinned host
buffers.  L2 is flushed (a 512 MB fill) before every timed step, outside the timed interval, because one step's
active weights (113 MB) would otherwise stay in the 126 MB L2.

`--impl reference` times the CPU oracle (a deliberately plain program) on a bounded sample of the same workload.
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
sys.path.insert(0, ROOT)

from paper_2609_19104_b200 import workloads as wl  # noqa: E402

METRIC = "masked_mlp_us_per_denoise_step"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per layer of a step, from ncu captures of the kernels that run these
# workloads (one layer launch of the lean per-layer kernel; the whole-step kernel's figure divided by its layers)
TRAFFIC_BYTES_PER_LAYER = {("pi0-stack-top25", 1): 6.794e6, ("pi0-stack-top25", 5): 6.62e6,
                           ("large-stack-top20-refresh2", 5): 42.7e6}
KERNEL_FAMILY = {0: "portable CUDA-core kernels (norm, gate/up, down)",
                 1: "fused_layer_kernel (lean per-layer cluster kernel, dependent-launch chained)",
                 2: "fused_layer_kernel, two tiles in flight",
                 3: "fused_layer_ws_kernel (warp-specialised per-layer cluster kernel)",
                 4: "stream_prep_kernel + stream_tile_kernel (per-layer streaming kernel)",
                 5: "step_kernel (whole step in one launch)"}


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def pick_workload(name: str) -> wl.Workload:
    if name == "config1":
        return wl.config1()
    if name == "config2":
        return wl.config2()
    if name == "config4":
        return wl.config4()
    if name == "config5":
        return wl.config5()
    if name.startswith("config6"):
        parts = name.split(":")
        return wl.config6(rho=float(parts[1]) if len(parts) > 1 else 0.25)
    if name.startswith("config3"):
        parts = name.split(":")
        rho = float(parts[1]) if len(parts) > 1 else 0.25
        B = int(parts[2]) if len(parts) > 2 else 1
        return wl.config3(rho, B=B)
    raise SystemExit(f"unknown workload {name}")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []                     # (host time, fields)
        self.proc = None
        self.t_begin = None

    def mark_begin(self):
        """The sampler is started before the warm-up so that nvidia-smi is already reporting; samples count from here."""
        self.t_begin = time.time()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20", "-i",
                 str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

        def summarise(rows):
            sm, mx, reasons = [], [], set()
            for _, r in rows:
                try:
                    sm.append(float(r[0]))
                    mx.append(float(r[1]))
                    for n, v in zip(names, r[2:6]):
                        if v.lower().startswith("active"):
                            reasons.add(n)
                except Exception:
                    continue
            return sm, mx, reasons

        # samples from the start of the timed steps to the end of the run (the side figures and the end-to-end steps
        # keep the GPU on the same work); a run too short for one such sample falls back to every sample taken
        # since the warm-up began, and says so
        window = "timed steps onward"
        sm, mx, reasons = summarise([x for x in self.rows if self.t_begin is None or x[0] >= self.t_begin])
        if not sm:
            window = "whole run including warm-up"
            sm, mx, reasons = summarise(self.rows)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "window": window}


# ------------------------------------------------------------------------------------------------ reference arm
def oracle_sample(w: wl.Workload, sample_layers: int):
    """Inputs of the bounded CPU sample: the first `sample_layers` layers of the stack, top-K lists drawn from the
    oracle's own dense records of those layers."""
    import oracle
    ws = wl.scaled(w, L=sample_layers)
    Wg, Wu, Wd = zip(*[wl.layer_weights(ws, l) for l in range(sample_layers)])
    r_ref = wl.bf16_bits_to_f32(wl.reference_input(w))
    _, rec = oracle.step(Wg, Wu, Wd, r_ref, return_records=True)
    idx = np.zeros((sample_layers, w.I), np.int32)
    cnt = np.zeros(sample_layers, np.int32)
    for l in range(sample_layers):
        s = oracle.compact_scores(rec[l], oracle.RULE_TOPK, k=w.K)
        idx[l, :s.size] = s
        cnt[l] = s.size
    return (Wg, Wu, Wd), idx, cnt


def time_oracle(w: wl.Workload, steps: int, warmup: int, sample_layers: int = 3):
    import oracle
    (Wg, Wu, Wd), idx, cnt = oracle_sample(w, sample_layers)
    scale_up = w.L / sample_layers
    times = []
    for s in range(warmup + steps):
        r0 = wl.bf16_bits_to_f32(wl.step_input(w, s % w.steps))
        t0 = time.perf_counter()
        oracle.step(Wg, Wu, Wd, r0, idx, cnt)
        dt = time.perf_counter() - t0
        if s >= warmup:
            times.append(dt)
    us = float(np.mean(times)) * 1e6 * scale_up
    return us, oracle.num_threads(), (f"{sample_layers} of {w.L} layers of one masked denoising step per timed step "
                                      f"(K={w.K} per layer), scaled by {scale_up:g}")


def time_oracle_config0_single_thread():
    """The small single-layer case (Bernoulli(0.30) mask on the config-1 layer shape) on one host thread."""
    import oracle
    w0 = wl.config0()
    Wg, Wu, Wd = wl.layer_weights(w0, 0)
    x, r = wl.step_input(w0, 0), wl.residual_input(w0)
    sel = np.flatnonzero(wl.bernoulli_mask(w0)).astype(np.int32)
    n = oracle.num_threads()
    oracle.set_threads(1)
    try:
        oracle.masked_mlp(x, Wg, Wu, Wd, r, sel)
        t0 = time.perf_counter()
        oracle.masked_mlp(x, Wg, Wu, Wd, r, sel)
        dt = time.perf_counter() - t0
    finally:
        oracle.set_threads(n)
    return dt * 1e6, int(sel.size)


def run_reference(args, w: wl.Workload):
    if rank_env()[1] != 0:                 # under a multi-rank launch rank 0 alone runs and prints
        return
    us, cores, sample = time_oracle(w, args.steps, args.warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64-accumulate/f32", "data": "synthetic",
        "config": {"workload": w.name, "L": w.L, "H": w.H, "I": w.I, "T": w.T, "K_per_layer": w.K},
        "cpu_baseline": {"value": us, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ ranks
# The path has no exchange step: N GPUs run N replicas of the model, each on its own episodes.  The only things the
# ranks share are the barrier around the timed region and the maximum of their device times.
def rank_env():
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def episodes_of_rank(rank: int, B: int):
    """Episode numbers (seeds of the synthetic inputs) rank `rank` works on: disjoint across ranks."""
    return list(range(rank * B, (rank + 1) * B))


def max_over_ranks(values, world: int, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank defines the job's time)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def job_us_per_step(total_ms: float, steps: int, world: int, B: int) -> float:
    """Whole-job metric: every rank ran `steps` steps of B episodes in `total_ms` (max over ranks)."""
    return total_ms * 1e3 / (steps * world * B)


# ------------------------------------------------------------------------------------------------ Context Cache
def measured_bf16_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


def run_context(args, w: wl.Workload):
    """The second workload (not the headline metric): one VLM FFN layer under the Context Cache.  A step = Eq. 2 drift
    scores, top-ceil(rho P) row selection, Eq. 3 recomputation of the selected rows and scatter."""
    import torch
    import paper_2609_19104_b200 as rm
    world, rank, local = rank_env()
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    P, S, H, I = w.extra["P"], w.extra["S"], w.H, w.I
    k = wl.topk_count(w.density, P)
    R = k + S
    ctx = rm.Context(1, H, I, T_max=64)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed + rank)
    mk = lambda shape: (torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32) * w.sigma).to(torch.bfloat16)
    Wg, Wu, Wd = mk((I, H)), mk((I, H)), mk((H, I))
    x_bits, xr_bits, y_ref = wl.context_inputs(w)
    to = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    x, xr, yref = to(x_bits), to(xr_bits), torch.from_numpy(y_ref).cuda()
    score = torch.empty(P, dtype=torch.float32, device="cuda")
    rows = torch.zeros(P, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    y_out = torch.empty(P + S, H, dtype=torch.float32, device="cuda")
    pin_x = torch.from_numpy(x_bits.view(np.int16)).pin_memory()
    pin_y = torch.empty(P + S, H, dtype=torch.float32).pin_memory()
    flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        ctx.rm_context_drift(x, xr, P, score)
        ctx.rm_mask_compact([score], rm.RM_SRC_SCORE_F32, rm.RM_REDUCE_TOPK, rows, cnt, P, n_lists=1, k=k, I=P)
        ctx.rm_context_ffn(Wg, Wu, Wd, x, rows, cnt, P, S, R, yref, y_out)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for s in range(args.warmup):
        flush.fill_(s & 0xFF)
        step()
    torch.cuda.synchronize()
    sampler.mark_begin()
    l0 = ctx.launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for s in range(args.steps):
        flush.fill_(s & 0xFF)
        ev[s][0].record(stream)
        step()
        ev[s][1].record(stream)
    torch.cuda.synchronize()
    launches = ctx.launch_count() - l0
    status = ctx.rm_device_status()
    if status != 0:
        raise RuntimeError(f"device status {status} ({rm.status_string(status)}) after the timed steps")
    total_ms = float(sum(a.elapsed_time(b) for a, b in ev))
    e2e = []
    for s in range(args.warmup + args.steps):
        flush.fill_(s & 0xFF)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        x.view(torch.int16).copy_(pin_x, non_blocking=True)
        step()
        pin_y.copy_(y_out, non_blocking=True)
        torch.cuda.synchronize()
        if s >= args.warmup:
            e2e.append(time.perf_counter() - t0)
    clocks = sampler.stop() if rank == 0 else None
    total_ms, e2e_ms = max_over_ranks([total_ms, float(sum(e2e)) * 1e3], world, device="cuda")
    if rank != 0:
        return
    us = total_ms * 1e3 / (args.steps * world)
    hbm_peak, kind = measured_hbm_peak()
    tf_peak, _ = measured_bf16_peak()
    flops = 2.0 * R * 3 * H * I
    bytes_step = 3 * H * I * 2 + (P + S) * H * 2 + P * H * 2 + 2 * R * H * 4 + 2 * R * I * 2
    achieved = bytes_step / (us * 1e-6) / 1e9
    line = {
        "metric": "context_cache_us_per_ffn_layer", "value": us, "unit": "us", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 (fp32 accumulate)", "data": "synthetic",
        "config": {"workload": w.name, "H": H, "I": I, "P": P, "S": S, "rows_recomputed": R,
                   "l2": "flushed before every timed step (512 MB fill, outside the timed interval)",
                   "multi_gpu": "replicas"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
                     "traffic": None, "peak_kind": f"{kind} copy bandwidth",
                     "kernel": "ctx_gemm_kernel (two launches: gate/up + GeLU, down with split K)",
                     "bytes_per_launch": bytes_step, "flops_per_step": flops,
                     "tensor_tflops": flops / (us * 1e-6) / 1e12, "tensor_frac_of_measured_bf16": flops / (us * 1e-6) / 1e12 / tf_peak,
                     "note": f"{R} rows against {3 * H * I / 1e6:.0f} M weights: {flops / bytes_step:.0f} flop/byte, at the ridge "
                             f"({tf_peak * 1e3 / hbm_peak:.0f} flop/byte)"},
        "e2e": {"value": e2e_ms * 1e3 / (args.steps * world), "unit": "us",
                "h2d_bytes_per_step": int(x_bits.nbytes), "d2h_bytes_per_step": int((P + S) * H * 4)},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    print(json.dumps(line))



# ------------------------------------------------------------------------------------------------ the other workloads
def side_configs(rm, ctx1, packed1, w1, flush, stream, args):
    """The workloads besides the headline one, measured in the same run and reported in the line's "configs" object:
    us per step (cold L2, CUDA events on the launching stream, median), algorithmic bytes per layer of a step,
    achieved GB/s and fraction of the measured copy bandwidth, and the kernel family the library chose by itself
    (read back from the library).  For batches the fraction is computed on the bytes that must leave HBM at least
    once -- the UNION of the episodes' lists -- and the sum over the episodes is given beside it."""
    import torch
    peak, _ = measured_hbm_peak()
    reps = max(5, min(args.steps, 20))
    f32 = lambda bits: torch.from_numpy(wl.bf16_bits_to_f32(bits))

    def timed_us(fn):
        evs = []
        for i in range(3 + reps):
            flush.fill_(i & 0xFF)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn(i)
            b.record(stream)
            if i >= 3:
                evs.append((a, b))
        torch.cuda.synchronize()
        return float(np.median([a.elapsed_time(b) for a, b in evs])) * 1e3

    def entry(ctx, w, us, K, B=1, union_rows=None, layers=None, note=None):
        L = w.L if layers is None else layers
        per_layer_sum = wl.algorithmic_bytes_per_layer(w.H, w.T, int(round(K))) * B
        e = {"us_per_step": us / B, "us_per_layer": us / L, "K_per_layer": K, "B": B, "T": w.T, "H": w.H, "I": w.I, "L": L,
             "kernel_family": ctx.rm_get_info("last_variant"), "kernel": KERNEL_FAMILY.get(ctx.rm_get_info("last_variant"))}
        if union_rows is None:
            e["bytes_per_layer"] = per_layer_sum
        else:
            act = per_layer_sum - int(round(K)) * 3 * w.H * 2 * B              # activations, residuals, indices of all episodes
            e["bytes_per_layer"] = int(union_rows * 3 * w.H * 2) + act
            e["bytes_per_layer_sum_over_episodes"] = per_layer_sum
            e["union_neurons_per_layer"] = union_rows
        e["achieved_gbs"] = e["bytes_per_layer"] * L / (us * 1e-6) / 1e9
        e["frac"] = e["achieved_gbs"] / peak
        if union_rows is not None:
            e["frac_on_sum_over_episodes"] = per_layer_sum * L / (us * 1e-6) / 1e9 / peak
        status = ctx.rm_device_status()
        if status != 0:
            raise RuntimeError(f"device status {status} in side workload {w.name}")
        if note:
            e["note"] = note
        return e

    def topk_lists(ctx, w, rec, K, n_lists):
        idx = torch.zeros(n_lists, w.I, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(n_lists, dtype=torch.int32, device="cuda")
        ctx.rm_mask_compact([rec.view(n_lists, w.I)], rm.RM_SRC_SCORE_F32, rm.RM_REDUCE_TOPK, idx, cnt, w.I, n_lists=n_lists, k=K)
        return idx, cnt

    out = {}
    # ---- config 3: density sweep and the batch of 8 on the headline model
    rec1 = torch.zeros(1, w1.L, w1.I, dtype=torch.float32, device="cuda")
    r_out = torch.empty(1, w1.T, w1.H, dtype=torch.float32, device="cuda")
    ref1 = f32(wl.reference_input(w1))[None].cuda()
    x1 = f32(wl.step_input(w1, 3))[None].cuda()
    ctx1.rm_action_expert_step(packed1, ref1, None, None, 0, r_out, records_out=rec1, B=1, T=w1.T)
    for rho in (0.2, 0.4, 1.0):
        w3 = wl.config3(rho)
        idx, cnt = topk_lists(ctx1, w3, rec1, w3.K, w3.L)
        ctx1.rm_set_option("count_hint", w3.K)
        us = timed_us(lambda i: ctx1.rm_action_expert_step(packed1, x1, idx, cnt, w3.I, r_out, B=1, T=w3.T))
        out[f"config3_rho{rho:g}"] = entry(ctx1, w3, us, w3.K)
    us = timed_us(lambda i: ctx1.rm_action_expert_step(packed1, x1, None, None, 0, r_out, records_out=rec1, B=1, T=w1.T))
    out["config1_dense_reference_step"] = entry(ctx1, w1, us, w1.I, note="idx = NULL, activation records emitted")
    B = 8
    w3b = wl.config3(0.25, B=B)
    ctxb = rm.Context(w3b.L, w3b.H, w3b.I, T_max=w3b.T, B_max=B)
    refs = torch.stack([f32(wl.reference_input(w3b, episode=b)) for b in range(B)]).cuda()
    xs = torch.stack([f32(wl.step_input(w3b, 2, episode=b)) for b in range(B)]).cuda()
    recb = torch.zeros(B, w3b.L, w3b.I, dtype=torch.float32, device="cuda")
    outb = torch.empty(B, w3b.T, w3b.H, dtype=torch.float32, device="cuda")
    ctxb.rm_action_expert_step(packed1, refs, None, None, 0, outb, records_out=recb, B=B, T=w3b.T)
    idxb, cntb = topk_lists(ctxb, w3b, recb, w3b.K, B * w3b.L)
    ctxb.rm_set_option("count_hint", w3b.K)
    h_idx = idxb.cpu().numpy().reshape(B, w3b.L, -1)
    union = float(np.mean([len(set().union(*[set(h_idx[b, l, :w3b.K].tolist()) for b in range(B)])) for l in range(w3b.L)]))
    us = timed_us(lambda i: ctxb.rm_action_expert_step(packed1, xs, idxb, cntb, w3b.I, outb, B=B, T=w3b.T))
    out["config3_rho0.25_B8"] = entry(ctxb, w3b, us, w3b.K, B=B, union_rows=union,
                                      note="us_per_step is per episode (one call runs 8 episodes); frac on the union of the lists")
    ctxb.close()
    # ---- config 4: T = 32, vote over a window of 4 records with a run-structured score scale
    w4 = wl.config4()
    ctx4 = rm.Context(w4.L, w4.H, w4.I, T_max=w4.T)
    scale = torch.from_numpy(np.stack([wl.run_structure(w4, l)[1] for l in range(w4.L)])).cuda()
    recs4 = []
    out4 = torch.empty(1, w4.T, w4.H, dtype=torch.float32, device="cuda")
    for i in range(w4.extra["window"]):
        rec = torch.zeros(1, w4.L, w4.I, dtype=torch.float32, device="cuda")
        ctx4.rm_action_expert_step(packed1, f32(wl.reference_input(w4, record=i))[None].cuda(), None, None, 0, out4,
                                   records_out=rec, record_scale=scale, B=1, T=w4.T)
        recs4.append(rec.view(w4.L, w4.I))
    idx4 = torch.zeros(w4.L, w4.I, dtype=torch.int32, device="cuda")
    cnt4 = torch.zeros(w4.L, dtype=torch.int32, device="cuda")
    ctx4.rm_mask_compact(recs4, rm.RM_SRC_SCORE_F32, rm.RM_REDUCE_TOPK, idx4, cnt4, w4.I, n_lists=w4.L, k=w4.K,
                         min_votes=w4.extra["min_votes"])
    K4 = float(cnt4.float().mean().item())
    ctx4.rm_set_option("count_hint", int(round(K4)))
    x4 = f32(wl.step_input(w4, 3))[None].cuda()
    us = timed_us(lambda i: ctx4.rm_action_expert_step(packed1, x4, idx4, cnt4, w4.I, out4, B=1, T=w4.T))
    out["config4"] = entry(ctx4, w4, us, K4, note="lists: 3-of-4 vote over per-record top-615 sets of run-structured records")
    ctx4.close()
    # ---- config 0: one layer, Bernoulli(0.30) mask, through rm_sparse_mlp
    w0 = wl.config0()
    ctx0 = rm.Context(1, w0.H, w0.I, T_max=w0.T)
    to = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    # eight copies of the layer in turn, so that consecutive timed calls do not find their weights in L2 either way
    g0, u0, d0 = wl.layer_weights(w0, 0)
    copies = [ctx0.rm_pack_weights(to(g0), to(u0), to(d0)) for _ in range(8)]
    mask = torch.from_numpy(wl.bernoulli_mask(w0)).cuda()
    idx0 = torch.zeros(w0.I, dtype=torch.int32, device="cuda")
    cnt0 = torch.zeros(1, dtype=torch.int32, device="cuda")
    ctx0.rm_mask_compact([mask], rm.RM_SRC_BOOL_U8, rm.RM_REDUCE_NONE, idx0, cnt0, w0.I, n_lists=1)
    K0 = int(cnt0.item())
    ctx0.rm_set_option("count_hint", K0)
    x0, r0 = to(wl.step_input(w0, 0)), torch.from_numpy(wl.residual_input(w0)).cuda()
    y0 = torch.empty(w0.T, w0.H, dtype=torch.float32, device="cuda")
    us = timed_us(lambda i: ctx0.rm_sparse_mlp(copies[i % 8], x0, r0, idx0, cnt0, y0, T=w0.T))
    out["config0_single_layer"] = entry(ctx0, w0, us, K0, layers=1, note="one rm_sparse_mlp call")
    ctx0.close()
    del copies
    # ---- config 2: H = 2048, I = 16384 (weights drawn on the device: 1.8 G values)
    w2 = wl.config2()
    ctx2 = rm.Context(w2.L, w2.H, w2.I, T_max=w2.T)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w2.seed)
    mk = lambda shape: (torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32) * w2.sigma).to(torch.bfloat16)
    packed2 = [ctx2.rm_pack_weights(mk((w2.I, w2.H)), mk((w2.I, w2.H)), mk((w2.H, w2.I))) for _ in range(w2.L)]
    rec2 = torch.zeros(1, w2.L, w2.I, dtype=torch.float32, device="cuda")
    out2 = torch.empty(1, w2.T, w2.H, dtype=torch.float32, device="cuda")
    xd = f32(wl.step_input(w2, 0))[None].cuda()
    xsp = f32(wl.step_input(w2, 1))[None].cuda()
    us_dense = timed_us(lambda i: ctx2.rm_action_expert_step(packed2, xd, None, None, 0, out2, records_out=rec2, B=1, T=w2.T))
    out["config2_dense_step"] = entry(ctx2, w2, us_dense, w2.I, note="even steps of the schedule: dense, activation records emitted")
    idx2, cnt2 = topk_lists(ctx2, w2, rec2, w2.K, w2.L)
    ctx2.rm_set_option("count_hint", w2.K)
    us_sparse = timed_us(lambda i: ctx2.rm_action_expert_step(packed2, xsp, idx2, cnt2, w2.I, out2, B=1, T=w2.T))
    e = entry(ctx2, w2, us_sparse, w2.K, note="odd steps of the schedule: masked with the previous step's top-20 % lists")
    e["traffic_bytes_per_layer"] = TRAFFIC_BYTES_PER_LAYER.get((w2.name, e["kernel_family"]))
    us_g = timed_us(lambda i: ctx2.rm_debug_gather_read_step(packed2, idx2, cnt2, w2.I))
    e["gather_read_microbench_us_per_step"] = us_g
    e["gather_read_microbench_gbs"] = w2.K * 3 * w2.H * 2 * w2.L / (us_g * 1e-6) / 1e9
    out["config2_sparse_step"] = e
    us_c = timed_us(lambda i: ctx2.rm_mask_compact([rec2.view(w2.L, w2.I)], rm.RM_SRC_SCORE_F32, rm.RM_REDUCE_TOPK, idx2, cnt2,
                                                   w2.I, n_lists=w2.L, k=w2.K))
    out["config2_schedule_10_steps"] = {"us_total": 5 * (us_dense + us_c + us_sparse), "mask_compact_us": us_c,
                                        "note": "5 x (dense step + top-k on the GPU + sparse step)"}
    ctx2.close()
    return out

# ------------------------------------------------------------------------------------------------ GPU arm
def run_gpu(args, w: wl.Workload):
    import torch
    import torch.distributed as dist
    import paper_2609_19104_b200 as rm

    world, rank, local = rank_env()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    B = w.B
    ctx = rm.Context(w.L, w.H, w.I, T_max=w.T, B_max=B)
    ctx.rm_set_option("count_hint", w.K)          # the lists hold K neurons: launch one cluster per 64-neuron tile
    if args.variant:
        ctx.rm_set_option("variant", args.variant)
    if args.max_clusters:
        ctx.rm_set_option("max_clusters", args.max_clusters)
    # weights: the workload's seeded draws (same on every rank: replicas of one model)
    packed = []
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    for l in range(w.L):
        if args.device_weights:
            # same distribution drawn on the device (seeded torch generator): for the large workloads, where the
            # host-side counter-based draws of 1.8 G weights would take minutes
            mk = lambda shape: (torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32) * w.sigma).to(torch.bfloat16)
            packed.append(ctx.rm_pack_weights(mk((w.I, w.H)), mk((w.I, w.H)), mk((w.H, w.I))))
        else:
            g, u, d = wl.layer_weights(w, l)
            to = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
            packed.append(ctx.rm_pack_weights(to(g), to(u), to(d)))
    torch.cuda.synchronize()

    # every rank runs its own episodes (replicas; no data-path collective)
    ep0 = episodes_of_rank(rank, B)[0]
    f32 = lambda bits: torch.from_numpy(wl.bf16_bits_to_f32(bits))
    refs = torch.stack([f32(wl.reference_input(w, episode=ep0 + b)) for b in range(B)]).cuda()
    step_inputs = [torch.stack([f32(wl.step_input(w, s, episode=ep0 + b)) for b in range(B)]) for s in range(w.steps)]
    dev_inputs = [t.cuda() for t in step_inputs]
    pinned_in = [t.pin_memory() for t in step_inputs]
    pinned_out = torch.empty(B, w.T, w.H, dtype=torch.float32).pin_memory()
    r_out = torch.empty(B, w.T, w.H, dtype=torch.float32, device="cuda")
    records = torch.zeros(B, w.L, w.I, dtype=torch.float32, device="cuda")
    idx = torch.zeros(B * w.L, w.I, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(B * w.L, dtype=torch.int32, device="cuda")
    n_lists = B * w.L
    rec_flat = records.view(n_lists, w.I)

    anchored = "group" in w.extra                 # the anchor schedule of Eq. 4 (dense anchor, then masked updates)
    if not anchored:
        # reference pass (dense, emits the activation records), then the masks
        ctx.rm_action_expert_step(packed, refs, None, None, 0, r_out, records_out=records, B=B, T=w.T)

        compact_layers = None
        if args.gather_once:
            if B != 1:
                raise SystemExit("--gather-once: compact layers are shared by the batch, so B must be 1")
            compact_layers = [torch.empty(ctx.packed_layer_bytes(), dtype=torch.uint8, device="cuda") for _ in range(w.L)]

        def compact():
            ctx.rm_mask_compact([rec_flat], rm.RM_SRC_SCORE_F32, rm.RM_REDUCE_TOPK, idx, cnt, w.I, n_lists=n_lists, k=w.K)
            if compact_layers is not None:
                for l in range(w.L):
                    ctx.rm_gather_weights(packed[l], idx[l], cnt[l:l + 1], w.I, compact_layers[l])
    else:
        # reference execution of all steps (one record per step), group masks by the group reduce (Sec. 5), anchor
        # state buffers and one output gate per step
        G = w.extra["group"]
        n_groups = w.steps // G
        step_recs = []
        for s in range(w.steps):
            ref_s = torch.stack([f32(wl.reference_step_input(w, s, episode=ep0 + b)) for b in range(B)]).cuda()
            rec_s = torch.zeros(B, w.L, w.I, dtype=torch.float32, device="cuda")
            ctx.rm_action_expert_step(packed, ref_s, None, None, 0, r_out, records_out=rec_s, B=B, T=w.T)
            step_recs.append(rec_s.view(n_lists, w.I))
        g_idx = [torch.zeros(n_lists, w.I, dtype=torch.int32, device="cuda") for _ in range(n_groups)]
        g_cnt = [torch.zeros(n_lists, dtype=torch.int32, device="cuda") for _ in range(n_groups)]
        idx, cnt = g_idx[0], g_cnt[0]
        h_stride = (w.T + 3) // 4 * 4
        y_an = torch.zeros(w.L, B, w.T, w.H, dtype=torch.float32, device="cuda")
        h_an = torch.zeros(w.L, B, w.I, h_stride, dtype=torch.float32, device="cuda")
        gates = [torch.stack([torch.from_numpy(wl.output_gate(w, s, episode=ep0 + b)) for b in range(B)], dim=1)
                 .contiguous().cuda() for s in range(w.steps)]                      # [L,B,H] per step

        def compact():
            for g in range(n_groups):
                ctx.rm_mask_compact(step_recs[g * G:(g + 1) * G], rm.RM_SRC_SCORE_F32, rm.RM_REDUCE_GROUP, g_idx[g],
                                    g_cnt[g], w.I, n_lists=n_lists, k=w.K)

    compact()
    torch.cuda.synchronize()
    K_mean = float(cnt.float().mean().item())

    def run_step(s, r_in):
        """One denoising step of the workload on device-resident input."""
        ss = s % w.steps
        if not anchored:
            if compact_layers is not None:
                ctx.rm_action_expert_step(compact_layers, r_in, None, cnt, 0, r_out, B=B, T=w.T)
            else:
                ctx.rm_action_expert_step(packed, r_in, idx, cnt, w.I, r_out, B=B, T=w.T)
        elif ss % G == 0:
            ctx.rm_action_expert_step_ex(packed, r_in, None, None, 0, r_out, rm.RM_ANCHOR_WRITE, y_an, h_an, h_stride,
                                         out_gate=gates[ss], B=B, T=w.T)
        else:
            ctx.rm_action_expert_step_ex(packed, r_in, g_idx[ss // G], g_cnt[ss // G], w.I, r_out, rm.RM_ANCHOR_UPDATE,
                                         y_an, h_an, h_stride, out_gate=gates[ss], B=B, T=w.T)

    flush = torch.empty(512 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def one_step(s, timed_events=None):
        flush.fill_(s & 0xFF)
        if timed_events is not None:
            timed_events[0].record(stream)
        if s % w.steps == 0:
            compact()
        run_step(s, dev_inputs[s % w.steps])
        if timed_events is not None:
            timed_events[1].record(stream)

    if args.phase_timeline:
        phase_timeline(ctx, w, lambda s: one_step(s))
        return
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for s in range(args.warmup):
        one_step(s)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()

    sampler.mark_begin()
    launches0 = ctx.launch_count()
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for s in range(args.steps):
        one_step(s, events[s])
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches = ctx.launch_count() - launches0
    step_variant = ctx.rm_get_info("last_variant")          # the kernel family the library chose for the timed steps
    status = ctx.rm_device_status()
    if status != 0:
        log = [ctx.rm_get_info(f"status_log:{i}") for i in range(ctx.rm_get_info("status_log_count"))]
        raise RuntimeError(f"device status {status} ({rm.status_string(status)}) after the timed steps; waits that gave "
                           f"up (source line, CTA): {[(d >> 12, d & 0xfff) for d in log]}: the timing is void")
    step_ms = [a.elapsed_time(b) for a, b in events]
    total_ms = float(sum(step_ms))

    # ---- side figures (outside the timed region of the headline): the same steps with a warm L2, the mask compaction
    # alone, and (plain workloads) the dense reference step with record emission
    def timed(fn, reps, flush_first):
        evs = []
        for i in range(reps):
            if flush_first:
                flush.fill_(i & 0xFF)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn(i)
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) * 1e3 for a, b in evs]

    warm_us = timed(lambda i: run_step(1 + i % (w.steps - 1), dev_inputs[(1 + i % (w.steps - 1)) % w.steps]), min(args.steps, 20), False)
    compact_us = timed(lambda i: compact(), 5, True)
    dense_us = None
    if not anchored:
        dense_us = timed(lambda i: ctx.rm_action_expert_step(packed, refs, None, None, 0, r_out, records_out=records, B=B, T=w.T),
                         3, True)
        compact()                                           # the lists again, from the records just rewritten
    # the same lists through the gather-read microbenchmark (layer by layer, cold L2): how fast they can leave HBM at all
    gather_us = timed(lambda i: ctx.rm_debug_gather_read_step(packed, idx, cnt, w.I), 5, True)
    union_rows = None
    if B > 1 and not anchored:
        h_idx, h_cnt = idx.cpu().numpy().reshape(B, w.L, -1), cnt.cpu().numpy().reshape(B, w.L)
        union_rows = float(np.mean([len(set().union(*[set(h_idx[b, l, :h_cnt[b, l]].tolist()) for b in range(B)]))
                                    for l in range(w.L)]))

    e2e_in = torch.empty(B, w.T, w.H, dtype=torch.float32, device="cuda")
    # end to end through the host-buffer entry point (H2D of the step input, step, D2H of the result, sync)
    e2e_times = []
    for s in range(args.warmup + args.steps):
        flush.fill_(s & 0xFF)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        if not anchored:
            ctx.rm_action_expert_step_host(packed, pinned_in[s % w.steps], idx, cnt, w.I, pinned_out, B=B, T=w.T)
        else:
            # the anchored step has no host-buffer entry point: the same three stages through the binding
            e2e_in.copy_(pinned_in[s % w.steps], non_blocking=True)
            run_step(s, e2e_in)
            pinned_out.copy_(r_out, non_blocking=True)
            torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        if s >= args.warmup:
            e2e_times.append(dt)
    e2e_total_ms = float(sum(e2e_times)) * 1e3

    # per-layer launch durations for the roofline: CUDA events around single-layer calls of the same kernels on the
    # same stream (cold L2 each time), layer by layer through the stack
    layer_ms = []
    x_bf16 = torch.empty(w.T, w.H, dtype=torch.bfloat16, device="cuda")
    y_tmp = torch.empty(w.T, w.H, dtype=torch.float32, device="cuda")
    res = dev_inputs[0][0].contiguous()
    x_bf16.copy_(res)
    reps = max(1, min(args.steps, 10))
    for rep in range(reps):
        for l in range(w.L):
            flush.fill_(l & 0xFF)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            ctx.rm_sparse_mlp(packed[l], x_bf16, res, idx[l], cnt[l:l + 1], y_tmp, T=w.T)
            b.record(stream)
            layer_ms.append((a, b))
    torch.cuda.synchronize()
    layer_us = float(np.mean([a.elapsed_time(b) for a, b in layer_ms])) * 1e3
    clocks = sampler.stop() if rank == 0 else None

    total_ms, e2e_total_ms = max_over_ranks([total_ms, e2e_total_ms], world, device="cuda")

    side = None
    if rank == 0 and world == 1 and w.config == 1 and not args.no_configs and not args.variant:
        side = side_configs(rm, ctx, packed, w, flush, stream, args)

    if rank == 0:
        us_per_step = job_us_per_step(total_ms, args.steps, world, B)   # per denoising step of one episode, whole job
        e2e_us = job_us_per_step(e2e_total_ms, args.steps, world, B)
        peak, peak_kind = measured_hbm_peak()
        if anchored:
            # average layer launch of the schedule: one dense anchor and G-1 masked updates per group
            bytes_layer = (wl.algorithmic_bytes_per_anchor_layer(w.H, w.T, w.I) +
                           (G - 1) * wl.algorithmic_bytes_per_update_layer(w.H, w.T, int(round(K_mean)))) // G * B
        else:
            bytes_layer = wl.algorithmic_bytes_per_layer(w.H, w.T, int(round(K_mean))) * B
        bytes_step = bytes_layer * w.L
        launches_per_step = launches / args.steps                 # fused layer launches + mask compaction share
        kernel_name = KERNEL_FAMILY.get(step_variant, f"variant {step_variant}")
        in_step_layer_us = us_per_step * B / w.L                  # average duration of a layer launch inside the step
        achieved = bytes_layer / (in_step_layer_us * 1e-6) / 1e9
        io_bytes = B * w.T * w.H * 4
        cpu_us, cores, sample = (time_oracle(w, steps=3, warmup=1) if world == 1 and not args.no_cpu_baseline and not anchored
                                 else (None, None, None))
        line = {
            "metric": METRIC, "value": us_per_step, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16 (fp32 accumulate)", "data": "synthetic",
            "config": {"workload": w.name, "L": w.L, "H": w.H, "I": w.I, "T": w.T, "B": B,
                       "K_per_layer": K_mean,
                       "mask": ("group masks (union of per-step top-k, ranked by summed score) of a reference execution, "
                                "rebuilt every 10 steps; schedule: dense anchor step, then 4 update steps (Eq. 4), gated"
                                if anchored else "top-k of dense reference records, rebuilt every 10 steps"
                                + (", rows copied to compact layers at every rebuild (gather-once)" if args.gather_once else "")),
                       "l2": "flushed before every timed step (512 MB fill, outside the timed interval)",
                       "multi_gpu": "replicas: each rank runs its own episodes, no collective on the data path"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": TRAFFIC_BYTES_PER_LAYER.get((w.name, step_variant)),
                         "peak_kind": f"{peak_kind} copy bandwidth", "kernel": kernel_name, "kernel_family": step_variant,
                         "bytes_per_launch": bytes_layer, "us_per_launch": in_step_layer_us,
                         "us_per_launch_isolated_cold": layer_us, "launches_per_step": launches_per_step,
                         "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS},
            "e2e": {"value": e2e_us, "unit": "us", "h2d_bytes_per_step": io_bytes, "d2h_bytes_per_step": io_bytes},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "per_step_us": {"median": float(np.median(step_ms)) * 1e3 / B, "p10": float(np.percentile(step_ms, 10)) * 1e3 / B,
                            "p90": float(np.percentile(step_ms, 90)) * 1e3 / B,
                            "note": "rank 0, per episode; the step that rebuilds the masks (one in ten) is the p90 tail"},
            "warm_l2_us_per_step": float(np.median(warm_us)) / B,
            "mask_compact_us": {"value": float(np.median(compact_us)), "lists": int(n_lists)},
            "gather_read_microbench": {
                "us_per_step": float(np.median(gather_us)),
                "gbs": int(round(K_mean)) * 3 * w.H * 2 * w.L / (float(np.median(gather_us)) * 1e-6) / 1e9,
                "note": "episode 0's lists of all layers read in ONE launch and discarded: one CTA per SM, whole 6H-byte rows by "
                        "16-byte cp.async, 12 rows in flight per CTA, cold L2: the rate at which these lists can leave HBM"},
        }
        if dense_us is not None:
            line["dense_step_us"] = float(np.median(dense_us)) / B
        if union_rows is not None:
            line["roofline"]["union_weight_bytes_per_launch"] = int(union_rows * 3 * w.H * 2)
            line["roofline"]["note"] = ("bytes_per_launch is the sum over the episodes' lists; the union of the lists (rows that "
                                        "must leave HBM at least once) is given beside it")
        if side is not None:
            line["configs"] = side
        if cpu_us is not None:
            line["cpu_baseline"] = {"value": cpu_us, "unit": "us", "cores": cores, "kind": "oracle", "sample": sample}
            us0, k0 = time_oracle_config0_single_thread()
            line["cpu_baseline"]["single_layer_one_thread_us"] = us0
            line["cpu_baseline"]["single_layer_one_thread_case"] = f"configs[0]: one layer, H=1024, I=4096, T=51, K={k0}"
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


PHASES = ["x ready (cluster barrier)", "first x stage landed, first gate/up product", "gate/up products complete",
          "h pieces sent", "first down product", "down products complete", "adds issued", "arrival on the counter",
          "counter complete: normalisation starts", "normalisation done"]
PHASE_ORDER = [8, 9, 0, 1, 2, 3, 4, 5, 6, 7]


def phase_timeline(ctx, w, step):
    """Profiling aid for a library built with -DRM_PHASE_TIMING=1 (python -m paper_2609_19104_b200.build with
    RM_EXTRA_NVCC_FLAGS set): runs three cold steps through the whole-step kernel and prints, per layer, when its
    phases were reached in the fastest and the slowest CTA (us after the first CTA saw the layer's counter complete)."""
    import ctypes
    import torch
    for s in range(1, 4):                                   # (step 0 of a schedule rebuilds the masks: skip it)
        step(s)
    torch.cuda.synchronize()
    if ctx.rm_get_info("last_variant") != 5:
        print(json.dumps({"phase_timeline": "the whole-step kernel did not run this workload"}))
        return
    n = 64 * 128 * 32
    buf = (ctypes.c_longlong * n)()
    rc = ctx.lib.rm_debug_phase_times(ctx._h, buf, -(1 << 20) - n)
    if rc != 0:
        print(json.dumps({"phase_timeline": f"unavailable (rm_debug_phase_times returned {rc}: build with -DRM_PHASE_TIMING=1)"}))
        return
    st = np.frombuffer(buf, dtype=np.int64).reshape(64, 128, 32).astype(np.float64)
    ncta = ctx.rm_get_info("persist_clusters") * 8
    t_first = None
    for it in range(min(w.L, 64)):
        s0 = st[it, :ncta, :10]
        go = s0[:, 8][s0[:, 8] > 0]
        ref = go.min() if go.size else s0[:, 1][s0[:, 1] > 0].min()
        t_first = ref if t_first is None else t_first
        row = {"layer": it, "starts_at_us": round((ref - t_first) / 1e3, 2)}
        for k in PHASE_ORDER:
            v = s0[:, k][s0[:, k] > 0]
            if v.size:
                row[PHASES[k]] = [round((v.min() - ref) / 1e3, 2), round((v.max() - ref) / 1e3, 2)]
        print(json.dumps(row))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config1")
    ap.add_argument("--device-weights", action="store_true",
                    help="draw the weights on the device with a seeded torch generator instead of the host generator")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--gather-once", action="store_true",
                    help="the paper's preparation of the weights: copy the masked rows into compact layers when the "
                         "masks are rebuilt (inside the timed region), then run the steps on the compact layers")
    ap.add_argument("--variant", type=int, default=0,
                    help="kernel variant override (library option \"variant\": 0 = chosen per launch)")
    ap.add_argument("--max-clusters", type=int, default=0, help="library option \"max_clusters\" (0 = default)")
    ap.add_argument("--layers", type=int, default=0,
                    help="run the first N layers of the workload only (small cases for profiler captures; not a bench value)")
    ap.add_argument("--phase-timeline", action="store_true",
                    help="profiling aid (library built with -DRM_PHASE_TIMING=1): print when each layer's phases were "
                         "reached inside the whole-step kernel, then exit; not a bench value")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the side measurements of the other workloads (the \"configs\" object of the line)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = pick_workload(args.workload)
    if args.layers > 0:
        w = wl.scaled(w, L=args.layers)
    if args.impl == "reference":
        run_reference(args, w)
    elif w.config == 6:
        run_context(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()
