#!/usr/bin/env python
"""Benchmark of the AdamA hot path on B200: fold / apply GB/s and fused wgrad+fold TFLOP/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload headline|gpt2xl|llama7b|sweep|small_tensors|extensions|oracle_timing|wgrad_shapes]

One step of the headline workload = one pass of the whole path:
  phase A  (flat 335M-parameter buffer, bf16 gradients, N=8):
           begin_minibatch, 8 x fold, apply
  phase B  (one 4096x4096 linear layer, 4096 tokens per micro-batch, N=4):
           begin_minibatch, 4 x linear_wgrad_fold, apply
All inputs are seeded synthetic tensors resident in HBM before the timed region.  Every
fold reads 6 GB and every fused call touches 335 MB, far more than the 126 MB L2, so
no L2 flush is needed between iterations.  Prints ONE JSON line.

`--impl reference` times the fp64 CPU oracle (plain C, as it stands) on a bounded sample
of the same workload on the host cores; it is a deliberately slow program, reported as a
baseline only.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import adama_workloads as wl  # noqa: E402

METRIC = "adama_fold_apply_wgrad_algorithmic_GBps"
UNIT = "GB/s"

FOLD_BYTES_BF16 = 18   # 2 B gradient + 8 B read m,v + 8 B write m,v
FOLD_BYTES_F32 = 20
APPLY_BYTES = 24       # read + write of w, m, v


def peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def step_bytes_and_flops(n_flat, n_micro_flat, tokens, d_in, d_out, n_micro_lin):
    """Algorithmic bytes and tensor flops of one headline step."""
    flat = n_flat * (FOLD_BYTES_BF16 * n_micro_flat + APPLY_BYTES)
    lin_params = d_in * d_out
    lin_call = 16 * lin_params + 2 * tokens * (d_in + d_out)
    lin = n_micro_lin * lin_call + APPLY_BYTES * lin_params
    flops = n_micro_lin * 2.0 * tokens * d_in * d_out
    return flat, lin, flops, lin_call


# ---- clocks ------------------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) != 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except (ValueError, IndexError):
            return local
    return local


# ---- the CPU oracle arm ------------------------------------------------------------------------

def oracle_sample_step(state):
    """One bounded sample of the headline step in the fp64 oracle (same flow, smaller sizes)."""
    import numpy as np
    import oracle
    flat, lin, grads, xs, ys = state["flat"], state["lin"], state["grads"], state["xs"], state["ys"]
    flat.begin_minibatch(len(grads))
    for g in grads:
        flat.fold(g)
    flat.update(wl.LR)
    lin.begin_minibatch(len(xs))
    for X, dY in zip(xs, ys):
        lin.fold(oracle.linear_wgrad(X, dY).reshape(-1))
    lin.update(wl.LR)
    return np  # keep numpy imported


def make_oracle_state(n_flat, tokens, d_in, d_out):
    import numpy as np
    import oracle
    from oracle import AdamAOracle
    f64 = lambda t: t.to(torch.float64).numpy()
    flat = AdamAOracle(f64(wl.normal((n_flat,), 0.02, torch.float32, wl.seed_for(2, 99))))
    grads = [f64(wl.normal((n_flat,), wl.CONFIG2.grad_std, torch.bfloat16, wl.seed_for(2, 0, i)))
             for i in range(wl.CONFIG2.n_micro)]
    lin = AdamAOracle(f64(wl.normal((d_in * d_out,), 0.02, torch.float32, wl.seed_for(3, 99))))
    xs = [f64(wl.normal((tokens, d_in), 1.0, torch.bfloat16, wl.seed_for(3, 0, i)))
          for i in range(wl.CONFIG3.n_micro)]
    ys = [f64(wl.normal((tokens, d_out), 1e-2, torch.bfloat16, wl.seed_for(3, 0, i) + 50))
          for i in range(wl.CONFIG3.n_micro)]
    return {"flat": flat, "lin": lin, "grads": grads, "xs": xs, "ys": ys,
            "threads": oracle.num_threads()}


# The bounded sample of the headline step that the oracle is timed on, in BOTH arms (the
# cpu_baseline of the default run and --impl reference): flat 2^24 parameters, linear layer
# 512 x 512 with 256 tokens.
ORACLE_SAMPLE = (1 << 24, 256, 512, 512)


def time_oracle(n_flat, tokens, d_in, d_out, steps, warmup, min_seconds=0.0):
    """Times `steps` sample steps (more, up to 50x, until `min_seconds` of work have run)."""
    state = make_oracle_state(n_flat, tokens, d_in, d_out)
    for _ in range(warmup):
        oracle_sample_step(state)
    t0 = time.perf_counter()
    done = 0
    while done < steps or (time.perf_counter() - t0 < min_seconds and done < 50 * steps):
        oracle_sample_step(state)
        done += 1
    dt = (time.perf_counter() - t0) / done
    flat_b, lin_b, flops, _ = step_bytes_and_flops(n_flat, wl.CONFIG2.n_micro, tokens, d_in, d_out,
                                                   wl.CONFIG3.n_micro)
    sample = (f"flat buffer of {n_flat} params (of {wl.CONFIG2_FULL_N}), N=8 bf16-valued grads; "
              f"linear layer {d_in}x{d_out}, {tokens} tokens (of 4096x4096, 4096), N=4; "
              "same flow, fp64, OpenMP over elements")
    return {"value": (flat_b + lin_b) / dt / 1e9, "unit": UNIT, "cores": state["threads"],
            "kind": "oracle", "sample": sample, "seconds_per_sample_step": dt, "sample_steps": done,
            "wgrad_gflops": flops / dt / 1e9}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    base = time_oracle(*ORACLE_SAMPLE, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": base["seconds_per_sample_step"] * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "headline (bounded sample per step): " + base["sample"]},
            "cpu_baseline": {k: base[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- our arm -----------------------------------------------------------------------------------

class EventTimer:
    """CUDA events recorded on torch's current stream (the stream every launch goes to)."""

    def __init__(self):
        self.marks = []

    def mark(self, label):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        self.marks.append((label, ev))

    def durations(self):
        """label -> list of ms between a mark and the next mark."""
        out = {}
        for (label, ev), (_, nxt) in zip(self.marks[:-1], self.marks[1:]):
            if label is not None:
                out.setdefault(label, []).append(ev.elapsed_time(nxt))
        return out


def run_ours(args):
    import paper_2305_19982_b200 as adama

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    pk = peaks()

    n = args.flat_params
    NA, NB = wl.CONFIG2.n_micro, wl.CONFIG3.n_micro
    T = args.linear_tokens
    d_in, d_out = args.linear_dims if args.linear_dims else (wl.CONFIG3.d_in, wl.CONFIG3.d_out)
    seed_shift = 100000 * rank  # each rank owns its own replica's data (weak scaling)

    # phase A state and inputs
    optA = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=local)
    w = wl.normal((n,), 0.02, torch.float32, wl.seed_for(2, 99) + seed_shift, device=dev)
    m = torch.zeros(n, device=dev)
    v = torch.zeros(n, device=dev)
    grads = [wl.normal((n,), wl.CONFIG2.grad_std, torch.bfloat16, wl.seed_for(2, 0, i) + seed_shift,
                       device=dev) for i in range(NA)]
    # phase B state and inputs
    optB = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=local)
    wB = wl.normal((d_in, d_out), 0.02, torch.float32, wl.seed_for(3, 99) + seed_shift, device=dev)
    mB = torch.zeros(d_in, d_out, device=dev)
    vB = torch.zeros(d_in, d_out, device=dev)
    Xs = [wl.normal((T, d_in), 1.0, torch.bfloat16, wl.seed_for(3, 0, i) + seed_shift, device=dev)
          for i in range(NB)]
    dYs = [wl.normal((T, d_out), 1e-2, torch.bfloat16, wl.seed_for(3, 0, i) + 50 + seed_shift,
                     device=dev) for i in range(NB)]

    # Data-parallel exchange at the end of each mini-batch (Section 3.3: the STATES are reduced,
    # once per mini-batch): "none" = independent replicas; "allreduce" = all-reduce of m and v,
    # then the update with the 1/R, 1/R^2 of Eqs. 6-7 folded in; "sharded" = reduce-scatter of
    # m and v, update of the owner's shard, all-gather of w.
    exchange = args.exchange if world > 1 else "none"
    if exchange != "none":
        from paper_2305_19982_b200 import ddp
    if exchange == "sharded" and (n % world or (d_in * d_out) % world):
        raise SystemExit("--exchange sharded needs buffer lengths that are multiples of the world size")

    def finish(opt, w_, m_, v_, label):
        if exchange == "allreduce":
            mark_ex(label + "_exchange")
            ddp.allreduce_states(m_, v_)
            mark_ex(label)
            opt.apply_allreduced(w_, m_, v_, wl.LR, world)
        elif exchange == "sharded":
            mark_ex(label + "_exchange")
            ddp.reduce_scatter_apply_allgather(opt, w_, m_, v_, wl.LR)
        else:
            mark_ex(label)
            opt.apply(w_, m_, v_, wl.LR)

    mark_ex = lambda label: None

    def step(timer=None):
        nonlocal mark_ex
        mark = timer.mark if timer else (lambda label: None)
        mark_ex = mark
        optA.begin_minibatch(NA)
        for i in range(NA):
            mark("fold")
            optA.fold(grads[i], m, v)
        finish(optA, w, m, v, "apply")
        optB.begin_minibatch(NB)
        for i in range(NB):
            mark("wgrad_fold")
            optB.linear_wgrad_fold(Xs[i], dYs[i], mB, vB)
        finish(optB, wB, mB, vB, "apply_linear")
        mark(None)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    launches0 = optA.launch_count + optB.launch_count
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    time.sleep(0.25)
    timer = EventTimer()
    barrier()
    start = torch.cuda.Event(enable_timing=True)
    stop = torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(args.steps):
        step(timer)
    stop.record()
    barrier()
    clocks = sampler.stop()
    total_ms = start.elapsed_time(stop)
    launches = optA.launch_count + optB.launch_count - launches0
    optA.sync_status()
    optB.sync_status()
    if dist is not None:
        t = torch.tensor([total_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps

    flat_b, lin_b, flops, lin_call_b = step_bytes_and_flops(n, NA, T, d_in, d_out, NB)
    value = world * (flat_b + lin_b) / (ms_per_step * 1e-3) / 1e9

    dur = timer.durations()
    avg = {k: sum(x) / len(x) for k, x in dur.items()}
    fold_gbs = FOLD_BYTES_BF16 * n / (avg["fold"] * 1e-3) / 1e9
    # (with --exchange sharded the update runs inside the exchange helper: no separate figure)
    apply_gbs = APPLY_BYTES * n / (avg["apply"] * 1e-3) / 1e9 if "apply" in avg else 0.0
    avg.setdefault("apply", 0.0)
    dur.setdefault("apply", [0.0])
    wgrad_tf = 2.0 * T * d_in * d_out / (avg["wgrad_fold"] * 1e-3) / 1e12
    roof_kernels = {
        "fold_bf16": {"bound": "hbm", "achieved": fold_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                      "frac": fold_gbs / pk["hbm_gbs"], "ms": avg["fold"],
                      "bytes_per_param": FOLD_BYTES_BF16, "params": n},
        "apply": {"bound": "hbm", "achieved": apply_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                  "frac": apply_gbs / pk["hbm_gbs"], "ms": avg["apply"],
                  "bytes_per_param": APPLY_BYTES, "params": n},
        "wgrad_fold": {"bound": "tensor", "achieved": wgrad_tf, "peak": pk["bf16_tflops"],
                       "unit": "TFLOP/s", "frac": wgrad_tf / pk["bf16_tflops"],
                       "frac_of_sustained": wgrad_tf / pk["bf16_tflops_sustained"],
                       "ms": avg["wgrad_fold"], "flops_per_call": 2.0 * T * d_in * d_out,
                       "hbm_bytes_per_call": lin_call_b, "traffic": None,
                       "hbm_gbs": lin_call_b / (avg["wgrad_fold"] * 1e-3) / 1e9},
    }
    traffic = load_traffic(n, T, d_in, d_out)
    for key in roof_kernels:
        roof_kernels[key]["traffic"] = traffic.get(key, {}).get("bytes_per_launch")
        roof_kernels[key]["traffic_note"] = traffic.get(key, {}).get("note")
    roofline = {"kernel": "fold_vec_kernel<bf16> (dominant: 8 launches per step)",
                "bound": "hbm", "achieved": fold_gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": fold_gbs / pk["hbm_gbs"], "peak_source": pk["source"],
                "traffic": traffic.get("fold_bf16", {}).get("bytes_per_launch"),
                "traffic_note": traffic.get("fold_bf16", {}).get("note")}

    # ---- end to end through the host-buffer entry points --------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(adama, dev, local, n, NA, NB, T, d_in, d_out, w, m, v, wB, mB, vB,
                      max(1, min(args.steps, 10)), flat_b + lin_b, world, dist)

    if "NCCL_DEBUG" in os.environ and rank == 0 and world > 1:
        sys.stderr.write(f"[bench] NCCL_DEBUG={os.environ['NCCL_DEBUG']}: communicator log above\n")

    # bytes each rank sends (= receives) per step in the exchange: ring all-reduce 2(R-1)/R of
    # the payload, reduce-scatter and all-gather (R-1)/R each
    params = n + d_in * d_out
    exchange_info = {"mode": exchange, "bytes_per_rank_per_step": 0}
    if exchange == "allreduce":
        exchange_info["bytes_per_rank_per_step"] = int(2 * (world - 1) / world * 8 * params)
        exchange_info["payload"] = "m and v, fp32 (8 B/param), one all-reduce each per mini-batch"
    elif exchange == "sharded":
        exchange_info["bytes_per_rank_per_step"] = int((world - 1) / world * 12 * params)
        exchange_info["payload"] = "reduce-scatter of m, v (8 B/param) + all-gather of w (4 B/param)"
    if exchange != "none":
        exchange_info["ms_per_step"] = (sum(dur.get("apply_exchange", [0.0])) +
                                        sum(dur.get("apply_linear_exchange", [0.0]))) / args.steps

    cpu_base = None
    peak_mem = None
    stacks = None
    if rank == 0:
        peak_mem = memory_report(adama, dev, local, T, d_in, d_out, Xs[0], dYs[0])
    optA.close()
    optB.close()
    del w, m, v, grads, wB, mB, vB, Xs, dYs
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_stacks:
        # the two layer-stack workloads in their stated configuration, 2 mini-batches each
        # ("_per_block": the linears of a transformer block folded by one grouped launch)
        # ("_settled": context flag ADAMA_INPUTS_SETTLED -- a call's operand loads do not wait for the
        # kernel before it; the stacks' inputs are complete long before, as the flag requires)
        stacks = {"gpt2xl": measure_stack("gpt2xl", 2, 1, dev_index=local),
                  "gpt2xl_per_block": measure_stack("gpt2xl", 2, 1, dev_index=local,
                                                    with_gemm_pipeline=False, layers_per_launch=4),
                  "gpt2xl_settled": measure_stack("gpt2xl", 2, 1, dev_index=local, with_gemm_pipeline=False,
                                                  inputs_settled=True, with_memory=False),
                  "gpt2xl_per_block_settled": measure_stack("gpt2xl", 2, 1, dev_index=local,
                                                            with_gemm_pipeline=False, layers_per_launch=4,
                                                            inputs_settled=True, with_memory=False)}
        free, _ = torch.cuda.mem_get_info()
        if free >= 100 * (1 << 30):
            stacks["llama7b"] = measure_stack("llama7b", 2, 1, dev_index=local)
            stacks["llama7b_per_block"] = measure_stack("llama7b", 2, 1, dev_index=local,
                                                        with_gemm_pipeline=False, layers_per_launch=7)
            stacks["llama7b_settled"] = measure_stack("llama7b", 2, 1, dev_index=local,
                                                      with_gemm_pipeline=False, inputs_settled=True,
                                                      with_memory=False)
        else:
            stacks["llama7b"] = {"skipped": f"needs ~90 GB of free device memory, {free >> 30} GiB free"}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            cpu_base = time_oracle(*ORACLE_SAMPLE, 2, 1, min_seconds=10.0)
            cpu_base = {k: cpu_base[k] for k in ("value", "unit", "cores", "kind", "sample",
                                                 "seconds_per_sample_step", "sample_steps")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 (bf16 inputs on the fused path)",
            "data": "synthetic",
            "config": {"workload": f"headline: flat {n}-param buffer (bf16 grads, N={NA}) fold+apply, "
                                   f"then linear {d_in}x{d_out} with {T} tokens (N={NB}) fused "
                                   "wgrad+fold + apply",
                       "l2": "inputs larger than L2, no flush", "replicas": world,
                       "exchange": exchange_info},
            "fold_apply_GBps": (flat_b / ((sum(dur["fold"]) + sum(dur["apply"])) / args.steps * 1e-3)) / 1e9,
            "wgrad_fold_TFLOPps": wgrad_tf,
            "roofline": roofline, "roofline_kernels": roof_kernels,
            "cpu_baseline": cpu_base, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks, "peak_memory": peak_mem, "stacks": stacks,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()  # rank 0 may still be printing; leave the group together
        dist.destroy_process_group()


def load_traffic(n_flat, tokens, d_in, d_out):
    """Per-launch DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) from the committed
    ncu summary (profiles/traffic.json: medians over the launches of a single-pass launch list of
    the bench's own full-size step).  A run on another buffer size scales the streaming kernels'
    figure by the element count (their traffic is proportional to it).  The fused call's entry
    counts only for the shape it was captured on.  An entry is dropped once one of the kernel's
    source files differs from those the counters were taken on."""
    import hashlib
    p = ROOT / "profiles" / "traffic.json"
    out = {}
    if not p.exists():
        return out
    try:
        data = json.loads(p.read_text())
    except ValueError:
        return out
    for key, ent in data.items():
        if not isinstance(ent, dict):
            continue
        srcs = [ROOT / f for f in ent.get("sources", [])]
        if not srcs or not all(f.is_file() for f in srcs):
            continue
        h = hashlib.sha256()
        for f in srcs:
            h.update(f.read_bytes())
        if h.hexdigest() != ent.get("sha256"):
            continue
        if "captured_params" in ent:
            scale = n_flat / ent["captured_params"]
            per_param = ent["captured_bytes"] / ent["captured_params"]
            note = (f"captured on launches of this size ({per_param:.2f} B/param)" if scale == 1.0 else
                    f"scaled by the element count from a {ent['captured_params']}-param capture "
                    f"({per_param:.2f} B/param)")
            out[key] = {"bytes_per_launch": int(ent["captured_bytes"] * scale), "note": note}
        elif ent.get("shape") == [tokens, d_in, d_out]:
            out[key] = {"bytes_per_launch": int(ent["captured_bytes"]),
                        "note": "captured on this shape"}
    return out


def run_e2e(adama, dev, local, n, NA, NB, T, d_in, d_out, w, m, v, wB, mB, vB, steps, step_bytes,
            world, dist):
    """The same step through the host-buffer entry points: every gradient, X and dY comes from
    pinned host memory and the updated weights are read back, all inside the timed region."""
    # copy-backs on the contexts' own streams: device-to-host traffic of one phase overlaps the
    # host-to-device traffic of the next (both directions of the link at once)
    optA = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=local, async_copyback=True)
    optB = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=local, async_copyback=True)
    g_host = [wl.normal((n,), wl.CONFIG2.grad_std, torch.bfloat16, 31 + i).pin_memory()
              for i in range(2)]
    X_host = wl.normal((T, d_in), 1.0, torch.bfloat16, 41).pin_memory()
    dY_host = wl.normal((T, d_out), 1e-2, torch.bfloat16, 42).pin_memory()
    w_host = torch.empty(n, dtype=torch.float32).pin_memory()
    wB_host = torch.empty(d_in * d_out, dtype=torch.float32).pin_memory()
    staging = torch.empty(max(256 << 20, 2 * T * (d_in + d_out) + 512), dtype=torch.uint8,
                          device=dev)

    def step():
        optA.begin_minibatch(NA)
        for i in range(NA):
            optA.fold_host(g_host[i & 1], m, v, staging)
        optA.apply_to_host(w, m, v, wl.LR, w_host)
        optB.begin_minibatch(NB)
        for i in range(NB):
            optB.linear_wgrad_fold_host(X_host, dY_host, mB, vB, staging)
        optB.apply_to_host(wB, mB, vB, wl.LR, wB_host)

    step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    start = torch.cuda.Event(enable_timing=True)
    stop = torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        step()
    # the last copy-backs belong to the timed region: make the stream wait for them first
    optA.sync_status()
    optB.sync_status()
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / steps
    if dist is not None:
        t = torch.tensor([ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    optA.close()
    optB.close()
    h2d = NA * n * 2 + NB * 2 * T * (d_in + d_out)
    d2h = 4 * n + 4 * d_in * d_out
    return {"value": world * step_bytes / (ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms,
            "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "api": "adama_fold_host / adama_linear_wgrad_fold_host / adama_apply_to_host "
                   "(contexts with ADAMA_ASYNC_COPYBACK)"}


def memory_report(adama, dev, local, T, d_in, d_out, X, dY):
    """Peak device memory of one micro-batch of the linear layer with the fused kernel (no
    gradient buffer) and with a materialised fp32 gradient folded by adama_fold."""
    opt = adama.AdamA(device=local)
    opt.begin_minibatch(1)
    mB = torch.zeros(d_in, d_out, device=dev)
    vB = torch.zeros(d_in, d_out, device=dev)
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats(dev)
    base = torch.cuda.memory_allocated(dev)
    opt.linear_wgrad_fold(X, dY, mB, vB)
    torch.cuda.synchronize()
    fused = torch.cuda.max_memory_allocated(dev) - base
    torch.cuda.reset_peak_memory_stats(dev)
    G = torch.empty(d_in, d_out, dtype=torch.float32, device=dev)  # the buffer AdamA's pipeline assigns
    try:
        torch.mm(X.t(), dY, out_dtype=torch.float32, out=G)
    except (TypeError, RuntimeError):
        G.zero_()  # the buffer is what is being measured, not its contents
    opt.fold(G.view(-1), mB.view(-1), vB.view(-1))
    torch.cuda.synchronize()
    mat = torch.cuda.max_memory_allocated(dev) - base
    del G
    opt.close()
    return {"layer": f"{d_in}x{d_out}", "extra_bytes_fused": int(fused),
            "extra_bytes_materialised_gradient": int(mat),
            "note": "bytes above the resident state and inputs during one micro-batch of the layer"}


def materialised_minibatch(stack, opt, n_micro, lr, inputs):
    """Comparison arm only, never the product path: the paper's own pipeline, in which every
    layer's fp32 weight gradient is assigned a buffer, filled by a library GEMM (cuBLAS through
    torch.mm), folded with adama_fold and released."""
    opt.begin_minibatch(n_micro)
    for i in range(n_micro):
        for j in reversed(range(len(stack.layers))):
            spec = stack.layers[j]
            X, dY = inputs(i, j, spec)
            G = torch.empty(spec.d_in, spec.d_out, dtype=torch.float32, device=stack.device)
            torch.mm(X.t(), dY, out_dtype=torch.float32, out=G)
            opt.fold(G.view(-1), stack.view(stack.m, j).view(-1), stack.view(stack.v, j).view(-1))
            del G
            if stack.biases:
                opt.bias_grad_fold(dY, stack.bias_view(stack.m, j), stack.bias_view(stack.v, j))
            del X, dY
    stack.apply(opt, lr)


def measure_stack(kind, steps, warmup, biases=False, with_gemm_pipeline=True, dev_index=0,
                  layers_per_launch=1, blocks=None, n_micro_override=None, inputs_settled=False,
                  with_memory=True):
    """GPT-2-XL- / Llama-7B-shaped stack, one mini-batch per step in the workload's own
    configuration (N = 8 / 16 micro-batches of 4096 tokens, layers back to front, fused
    weight-gradient fold per layer, one apply): time, TFLOP/s of the whole mini-batch, clocks,
    peak device memory without a gradient buffer, with a per-layer one and with a whole-model one.
    layers_per_launch > 1: that many consecutive layers (a transformer block's linears) are folded
    by one grouped launch, their X, dY released together after it.
    inputs_settled: the context is created with ADAMA_INPUTS_SETTLED (the pooled X, dY are complete
    long before any call, which is what the flag promises)."""
    import paper_2305_19982_b200 as adama
    from paper_2305_19982_b200.stack import gpt2xl_stack, llama7b_stack

    dev = torch.device("cuda", dev_index)
    pk = peaks()
    if kind == "gpt2xl":
        stack, tokens, n_micro, cfg_id = (gpt2xl_stack(blocks or wl.CONFIG4_BLOCKS, device=dev, biases=biases),
                                          wl.CONFIG4_TOKENS, wl.CONFIG4_N_MICRO, 4)
    else:
        stack, tokens, n_micro, cfg_id = (llama7b_stack(blocks or wl.CONFIG5_BLOCKS, device=dev),
                                          wl.CONFIG5_TOKENS, wl.CONFIG5_N_MICRO, 5)
    n_micro = n_micro_override or n_micro
    stack.w.normal_(0, 0.02, generator=torch.Generator(device=dev).manual_seed(wl.seed_for(cfg_id, 99)))
    # two seeded variants of X and dY per distinct width, reused across layers while timing
    widths = sorted({L.d_in for L in stack.layers} | {L.d_out for L in stack.layers})
    pool_x = {d: [wl.normal((tokens, d), 1.0, torch.bfloat16, wl.seed_for(cfg_id, 0, k) + d, device=dev)
                  for k in range(2)] for d in widths}
    pool_y = {d: [wl.normal((tokens, d), 1e-2, torch.bfloat16, wl.seed_for(cfg_id, 0, k) + 50 + d, device=dev)
                  for k in range(2)] for d in widths}
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=dev_index, inputs_settled=inputs_settled)

    def pooled(i, j, spec):
        return pool_x[spec.d_in][(i + j) & 1], pool_y[spec.d_out][(i + j) & 1]

    for _ in range(max(1, warmup)):
        stack.minibatch(opt, n_micro, wl.LR, pooled, layers_per_launch)
    torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(dev_index))
    sampler.start()
    launches0 = opt.launch_count
    start = torch.cuda.Event(enable_timing=True)
    stop = torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        stack.minibatch(opt, n_micro, wl.LR, pooled, layers_per_launch)
    stop.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = start.elapsed_time(stop) / steps
    launches = opt.launch_count - launches0
    opt.sync_status()
    flops = n_micro * stack.flops_per_micro_batch(tokens)
    tf = flops / (ms * 1e-3) / 1e12
    ms_layer = None
    if with_gemm_pipeline:
        # the paper's pipeline (per-layer gradient assigned, folded, released) for comparison
        materialised_minibatch(stack, opt, n_micro, wl.LR, pooled)
        torch.cuda.synchronize()
        s2 = torch.cuda.Event(enable_timing=True)
        e2 = torch.cuda.Event(enable_timing=True)
        s2.record()
        materialised_minibatch(stack, opt, n_micro, wl.LR, pooled)
        e2.record()
        torch.cuda.synchronize()
        ms_layer = s2.elapsed_time(e2)

    # peak memory: fresh X, dY per layer (as a backward pass would hand them over)
    def fresh(i, j, spec):
        return (torch.empty(tokens, spec.d_in, dtype=torch.bfloat16, device=dev).fill_(0.5),
                torch.empty(tokens, spec.d_out, dtype=torch.bfloat16, device=dev).fill_(0.01))

    del pool_x, pool_y
    torch.cuda.empty_cache()
    mem = {}
    for mode in (("none", "layer") if with_memory else ()):
        torch.cuda.synchronize()
        torch.cuda.reset_peak_memory_stats(dev)
        if mode == "none":
            stack.minibatch(opt, 1, wl.LR, fresh, layers_per_launch)
        else:
            materialised_minibatch(stack, opt, 1, wl.LR, fresh)
        torch.cuda.synchronize()
        mem[mode] = int(torch.cuda.max_memory_allocated(dev))
    opt.sync_status()
    state_bytes = 3 * 4 * stack.numel
    largest_layer = max(L.d_in * L.d_out for L in stack.layers)
    out = {
        "workload": kind, "biases": bool(stack.biases), "layers": len(stack.layers),
        "params": stack.n_params, "tokens_per_micro_batch": tokens, "n_micro": n_micro,
        "layers_per_launch": layers_per_launch, "inputs_settled_flag": bool(inputs_settled),
        "steps": steps, "ms_per_minibatch": ms, "TFLOPps": tf,
        "frac_of_sustained_bf16": tf / pk["bf16_tflops_sustained"],
        "frac_of_burst_bf16": tf / pk["bf16_tflops"], "peak_source": pk["source"],
        "gpu_launches": int(launches), "clocks": clocks,
        "gemm_plus_fold_pipeline_ms_per_minibatch": ms_layer,
        "peak_memory": None if not with_memory else {
            "state_bytes": state_bytes,
            "fused_no_gradient_buffer": mem["none"],
            "per_layer_gradient_released": mem["layer"],
            "whole_model_gradient_accumulation": mem["none"] + 4 * stack.n_params,
            "largest_layer_gradient_bytes": 4 * largest_layer,
            "note": "max_memory_allocated over one micro-batch with fresh X, dY per layer; "
                    "the gradient-accumulation figure adds an fp32 gradient for every parameter"},
    }
    opt.close()
    del stack
    torch.cuda.empty_cache()
    return out


def run_stack(args):
    """One stack workload on its own (python bench.py --workload gpt2xl|llama7b)."""
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(0)
    r = measure_stack(args.workload, args.steps, min(args.warmup, 2), biases=args.biases,
                      layers_per_launch=args.layers_per_launch, blocks=args.stack_blocks,
                      n_micro_override=args.stack_micro, with_gemm_pipeline=not args.stack_blocks,
                      inputs_settled=args.inputs_settled)
    pk = peaks()
    line = {
        "metric": "adama_wgrad_fold_stack_TFLOPps", "value": r["TFLOPps"], "unit": "TFLOP/s", "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": r["ms_per_minibatch"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 inputs, f32 accumulate and state", "data": "synthetic",
        "config": {"workload": args.workload, "biases": r["biases"], "layers": r["layers"],
                   "params": r["params"], "tokens_per_micro_batch": r["tokens_per_micro_batch"],
                   "n_micro": r["n_micro"], "layers_per_launch": r["layers_per_launch"],
                   "l2": "inputs larger than L2, no flush"},
        "roofline": {"kernel": "wgrad_fold_kernel", "bound": "tensor", "achieved": r["TFLOPps"],
                     "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": r["frac_of_sustained_bf16"], "frac_of_burst": r["frac_of_burst_bf16"],
                     "peak_source": pk["source"] + " (sustained)", "traffic": None},
        "materialised_per_layer_ms_per_step": r["gemm_plus_fold_pipeline_ms_per_minibatch"],
        "peak_memory": r["peak_memory"],
        "cpu_baseline": None, "e2e": None, "gpu_launches": r["gpu_launches"], "clocks": r["clocks"],
    }
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Config 2's size sweep: fold (bf16 g) and apply at 2^20 .. 2^28 and 335 M elements;
    median and best of 30 launches each, L2 flushed before every launch for sizes that
    would otherwise stay L2-resident."""
    import paper_2305_19982_b200 as adama
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pk = peaks()
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=0)
    opt.begin_minibatch(wl.CONFIG2.n_micro)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    rows = []
    for n in wl.CONFIG2_SWEEP:
        w = wl.normal((n,), 0.02, torch.float32, 1, device=dev)
        m = torch.zeros(n, device=dev)
        v = torch.zeros(n, device=dev)
        g = wl.normal((n,), wl.CONFIG2.grad_std, torch.bfloat16, 2, device=dev)
        res = {"n": n}
        for name, call, bpp in (("fold", lambda: opt.fold(g, m, v), FOLD_BYTES_BF16),
                                ("apply", lambda: opt.apply(w, m, v, wl.LR), APPLY_BYTES)):
            for _ in range(3):
                call()
            ts = []
            for _ in range(30):
                flush.zero_()
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                e0.record()
                call()
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            ts.sort()
            med, best = ts[len(ts) // 2], ts[0]
            res[name] = {"us_median": med * 1e3, "us_best": best * 1e3,
                         "GBps_median": bpp * n / (med * 1e-3) / 1e9,
                         "frac_of_peak": bpp * n / (med * 1e-3) / 1e9 / pk["hbm_gbs"]}
        rows.append(res)
        del w, m, v, g
    print(json.dumps({"metric": "adama_fold_apply_size_sweep", "unit": "GB/s", "peak": pk["hbm_gbs"],
                      "peak_source": pk["source"], "l2": "flushed before every launch",
                      "rows": rows}), flush=True)
    opt.close()


def run_extensions(args):
    """The kernels beside the headline path at the flat workload's size (335 M elements, inputs far
    above the L2): the fold with fp32 gradients, SGD-momentum fold / apply, the coefficient
    statistics, apply with the bf16 copy.  Median of 20 launches each, CUDA events, against the same HBM peak."""
    import paper_2305_19982_b200 as adama
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pk = peaks()
    n = wl.CONFIG2_FULL_N
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=0)
    opt.begin_minibatch(wl.CONFIG2.n_micro)
    w = wl.normal((n,), 0.02, torch.float32, 1, device=dev)
    m = wl.normal((n,), 1e-4, torch.float32, 3, device=dev)
    m0 = wl.normal((n,), 1e-4, torch.float32, 4, device=dev)
    v = wl.normal((n,), 1e-4, torch.float32, 5, device=dev).square_()
    va = v.clone()
    g = wl.normal((n,), wl.CONFIG2.grad_std, torch.bfloat16, 2, device=dev)
    wb = torch.empty(n, dtype=torch.bfloat16, device=dev)
    stats = torch.zeros(4, dtype=torch.float64, device=dev)
    rows = {}
    g32 = wl.normal((n,), wl.CONFIG2.grad_std, torch.float32, 6, device=dev)
    for name, call, bpp in (
            ("fold_f32_gradients", lambda: opt.fold(g32, m, v), 20),
            ("sgdm_fold_bf16", lambda: opt.sgdm_fold(g, m), 2 + 8),
            ("sgdm_apply", lambda: opt.sgdm_apply(w, m, 1e-3, 0.9), 16),
            ("coefficient_stats", lambda: opt.coefficient_stats(m, m0, v, va, stats), 20),
            ("apply_bf16_copy", lambda: opt.apply_bf16_copy(w, m, v, wb, wl.LR), 26)):
        for _ in range(3):
            call()
        ts = []
        for _ in range(20):
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            call()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ts.sort()
        med = ts[len(ts) // 2]
        rows[name] = {"ms_median": med, "ms_best": ts[0], "bytes_per_param": bpp,
                      "GBps_median": bpp * n / (med * 1e-3) / 1e9,
                      "frac_of_peak": bpp * n / (med * 1e-3) / 1e9 / pk["hbm_gbs"]}
    print(json.dumps({"metric": "adama_extension_kernels", "unit": "GB/s", "params": n,
                      "peak": pk["hbm_gbs"], "peak_source": pk["source"],
                      "l2": "inputs larger than L2, no flush", "rows": rows}), flush=True)
    opt.close()


def run_oracle_timing(args):
    """The oracle's own kernels timed on the host cores, with 1 thread and with all of them: fold
    and update at 2^20 and 2^24 elements (M params/s and effective GB/s at 18 and 24 B/param, the
    GPU kernels' byte counts), the naive weight gradient at 1024^3 (GFLOP/s).  A baseline beside
    the GPU numbers, nothing more; the oracle is timed as it stands."""
    import platform

    import numpy as np

    import oracle
    all_threads = oracle.num_threads()
    rows = []
    rng = np.random.default_rng(0)
    for threads in sorted({1, all_threads}):
        oracle.set_num_threads(threads)
        for n in (1 << 20, 1 << 24):
            orc = oracle.AdamAOracle(rng.normal(0, 0.02, n), wl.BETA1, wl.BETA2, wl.EPS)
            g = rng.normal(0, 1e-3, n)
            orc.begin_minibatch(8)
            reps = 20 if n <= (1 << 20) else 3
            orc.fold(g)
            t0 = time.perf_counter()
            for _ in range(reps):
                orc.fold(g)
            tf = (time.perf_counter() - t0) / reps
            orc.update(wl.LR)
            t0 = time.perf_counter()
            for _ in range(reps):
                orc.update(wl.LR)
            tu = (time.perf_counter() - t0) / reps
            rows.append({"threads": threads, "n": n,
                         "fold_Mparams_per_s": n / tf / 1e6, "fold_GBps_at_18B": 18 * n / tf / 1e9,
                         "update_Mparams_per_s": n / tu / 1e6,
                         "update_GBps_at_24B": 24 * n / tu / 1e9})
        d = 1024
        X = rng.normal(0, 1, (d, d))
        dY = rng.normal(0, 1e-2, (d, d))
        t0 = time.perf_counter()
        oracle.linear_wgrad(X, dY)
        tg = time.perf_counter() - t0
        rows.append({"threads": threads, "wgrad": "1024^3", "seconds": tg,
                     "GFLOPps": 2.0 * d ** 3 / tg / 1e9})
    oracle.set_num_threads(all_threads)
    cpu = platform.processor() or platform.machine()
    try:
        for ln in open("/proc/cpuinfo"):
            if ln.startswith("model name"):
                cpu = ln.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    print(json.dumps({"metric": "adama_oracle_host_timing", "kind": "oracle", "cores": all_threads,
                      "cpu": cpu, "rows": rows}), flush=True)


def run_wgrad_shapes(args):
    """The fused weight-gradient call on every distinct layer shape of the workloads (4096 tokens),
    alone, with the bias gradient folded in the same launch, and followed by the separate bias
    kernel; timed back to back and one call at a time with the L2 flushed."""
    import paper_2305_19982_b200 as adama
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pk = peaks()
    T = wl.CONFIG3.tokens
    shapes = [(wl.CONFIG3.d_in, wl.CONFIG3.d_out)]
    for _, di, do in list(wl.llama7b_block_linears()) + list(wl.gpt2xl_block_linears()):
        if (di, do) not in shapes:
            shapes.append((di, do))
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=0)
    opt.begin_minibatch(4)
    # a second context with ADAMA_INPUTS_SETTLED: a call's operand loads do not wait for the kernel
    # before it (X, dY below are complete long before any call, as the flag requires)
    opt_s = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=0, inputs_settled=True)
    opt_s.begin_minibatch(4)

    def timed(call, reps=20):
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e3

    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)

    def timed_cold(call, reps=10):
        # one call at a time with the L2 overwritten before it: what a layer costs inside a model
        # whose states are far larger than the L2
        ts = []
        for _ in range(reps):
            flush.zero_()
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            call()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        ts.sort()
        return ts[len(ts) // 2]

    def timed_in_model(d_in, d_out, make_call, reps=3):
        # as inside a model: calls back to back, each on its own copy of the layer's m and v, enough
        # copies that a call never finds its states in the L2 (>= 640 MB of states in the cycle);
        # no launch bubble as around a single call, no warm L2 as with one buffer
        copies = max(2, -(-(640 << 20) // (8 * d_in * d_out)))
        states = [(torch.zeros(d_in, d_out, device=dev), torch.zeros(d_in, d_out, device=dev))
                  for _ in range(copies)]
        for mm, vv in states:
            make_call(mm, vv)
        torch.cuda.synchronize()
        time.sleep(0.5)
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for mm, vv in states:
                make_call(mm, vv)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (reps * copies) * 1e3

    rows = []
    for d_in, d_out in shapes:
        X = wl.normal((T, d_in), 1.0, torch.bfloat16, 1, device=dev)
        dY = wl.normal((T, d_out), 1e-2, torch.bfloat16, 2, device=dev)
        m = torch.zeros(d_in, d_out, device=dev)
        v = torch.zeros(d_in, d_out, device=dev)
        mb = torch.zeros(d_out, device=dev)
        vb = torch.zeros(d_out, device=dev)

        def both():
            opt.linear_wgrad_fold(X, dY, m, v)
            opt.bias_grad_fold(dY, mb, vb)

        def rested(fn, call):
            # a pause before every measurement: under the power cap the SM clock sags after a few
            # milliseconds of dense tensor work and would carry over into the next shape
            torch.cuda.synchronize()
            time.sleep(0.5)
            return fn(call)

        us = rested(timed, lambda: opt.linear_wgrad_fold(X, dY, m, v))
        us_fused = rested(timed, lambda: opt.linear_wgrad_fold(X, dY, m, v, mb, vb))
        us_sep = rested(timed, both)
        cold = rested(timed_cold, lambda: opt.linear_wgrad_fold(X, dY, m, v))
        cold_fused = rested(timed_cold, lambda: opt.linear_wgrad_fold(X, dY, m, v, mb, vb))
        cold_sep = rested(timed_cold, both)
        tf = 2.0 * T * d_in * d_out / us / 1e6
        tf_cold = 2.0 * T * d_in * d_out / cold / 1e6
        us_model = timed_in_model(d_in, d_out, lambda mm, vv: opt.linear_wgrad_fold(X, dY, mm, vv))
        tf_model = 2.0 * T * d_in * d_out / us_model / 1e6
        us_set = timed_in_model(d_in, d_out, lambda mm, vv: opt_s.linear_wgrad_fold(X, dY, mm, vv))
        tf_set = 2.0 * T * d_in * d_out / us_set / 1e6
        rows.append({"d_in": d_in, "d_out": d_out, "tokens": T,
                     "in_model": {"us": us_model, "TFLOPps": tf_model,
                                  "frac_of_burst_peak": tf_model / pk["bf16_tflops"],
                                  "frac_of_sustained_peak": tf_model / pk["bf16_tflops_sustained"]},
                     "in_model_inputs_settled": {"us": us_set, "TFLOPps": tf_set,
                                                 "frac_of_burst_peak": tf_set / pk["bf16_tflops"],
                                                 "frac_of_sustained_peak": tf_set / pk["bf16_tflops_sustained"]},
                     "back_to_back": {"us": us, "TFLOPps": tf,
                                      "frac_of_burst_peak": tf / pk["bf16_tflops"],
                                      "us_with_fused_bias": us_fused,
                                      "us_with_separate_bias_kernel": us_sep},
                     "l2_flushed": {"us": cold, "TFLOPps": tf_cold,
                                    "frac_of_burst_peak": tf_cold / pk["bf16_tflops"],
                                    "us_with_fused_bias": cold_fused,
                                    "us_with_separate_bias_kernel": cold_sep}})
        del X, dY, m, v
    # token sweep on the 4096 x 4096 layer: below ~2000 tokens the call is bound by the 16 B/param
    # of m, v traffic, above by the tensor cores
    sweep = []
    d_in, d_out = wl.CONFIG3.d_in, wl.CONFIG3.d_out
    m = torch.zeros(d_in, d_out, device=dev)
    v = torch.zeros(d_in, d_out, device=dev)
    for tokens in (256, 512, 1024, 2048, 4096, 8192):
        X = wl.normal((tokens, d_in), 1.0, torch.bfloat16, 3, device=dev)
        dY = wl.normal((tokens, d_out), 1e-2, torch.bfloat16, 4, device=dev)
        torch.cuda.synchronize()
        time.sleep(0.5)
        us = timed_cold(lambda: opt.linear_wgrad_fold(X, dY, m, v))
        us_model = timed_in_model(d_in, d_out, lambda mm, vv: opt.linear_wgrad_fold(X, dY, mm, vv))
        byts = 16 * d_in * d_out + 2 * tokens * (d_in + d_out)
        sweep.append({"tokens": tokens, "us": us, "TFLOPps": 2.0 * tokens * d_in * d_out / us / 1e6,
                      "hbm_GBps": byts / us / 1e3,
                      "in_model_us": us_model, "in_model_hbm_GBps": byts / us_model / 1e3,
                      "in_model_frac_of_hbm_peak": byts / us_model / 1e3 / pk["hbm_gbs"],
                      "in_model_TFLOPps": 2.0 * tokens * d_in * d_out / us_model / 1e6,
                      "hbm_floor_us": byts / pk["hbm_gbs"] / 1e3,
                      "tensor_floor_us": 2.0 * tokens * d_in * d_out / pk["bf16_tflops"] / 1e6})
        del X, dY
    # the linears of one transformer block folded by ONE grouped launch (adama_linear_wgrad_fold_multi),
    # back to front, timed like "in_model" over enough copies of the block's states
    blocks = []
    for name, linears in (("gpt2xl_block", list(wl.gpt2xl_block_linears())),
                          ("llama7b_block", list(wl.llama7b_block_linears()))):
        linears = linears[::-1]
        state_bytes = sum(8 * di * do for _, di, do in linears)
        copies = max(2, -(-(640 << 20) // state_bytes))
        xs = {d: wl.normal((T, d), 1.0, torch.bfloat16, 5 + d, device=dev) for d in {di for _, di, _ in linears}}
        ys = {d: wl.normal((T, d), 1e-2, torch.bfloat16, 6 + d, device=dev) for d in {do for _, _, do in linears}}
        groups = [[(xs[di], ys[do], torch.zeros(di, do, device=dev), torch.zeros(di, do, device=dev))
                   for _, di, do in linears] for _ in range(copies)]
        res = {}
        for mode in ("one_launch_per_block", "one_launch_per_layer",
                     "one_launch_per_block_inputs_settled", "one_launch_per_layer_inputs_settled"):
            o = opt_s if mode.endswith("_inputs_settled") else opt

            def run(g):
                if mode.startswith("one_launch_per_block"):
                    o.linear_wgrad_fold_multi(g)
                else:
                    for item in g:
                        o.linear_wgrad_fold(*item)
            for g in groups:
                run(g)
            torch.cuda.synchronize()
            time.sleep(0.5)
            reps = 3
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                for g in groups:
                    run(g)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) / (reps * copies) * 1e3
            tf = sum(2.0 * T * di * do for _, di, do in linears) / us / 1e6
            res[mode] = {"us_per_block": us, "TFLOPps": tf, "frac_of_burst_peak": tf / pk["bf16_tflops"],
                         "frac_of_sustained_peak": tf / pk["bf16_tflops_sustained"]}
        blocks.append({"block": name, "layers": [[di, do] for _, di, do in linears], "tokens": T, **res})
        del groups, xs, ys
    opt.sync_status()
    opt_s.sync_status()
    opt_s.close()
    print(json.dumps({"metric": "adama_wgrad_fold_per_shape", "token_sweep_4096x4096_l2_flushed": sweep,
                      "blocks_in_model": blocks, "unit": "us", "peak_tflops": pk["bf16_tflops"],
                      "peak_source": pk["source"],
                      "timing": "back_to_back: 20 calls between two CUDA events (buffers may stay in "
                                "the L2); l2_flushed: median of 10 single calls, 512 MB written before each; "
                                "in_model: calls back to back, each on its own copy of m and v, >= 640 MB of "
                                "states in the cycle (cold L2, no single-call launch bubble)",
                      "rows": rows}), flush=True)
    opt.close()


def run_small_tensors(args):
    """The non-matrix parameters of a GPT-2-XL-shaped model (per block: two norms, four biases;
    432 tensors, 1.0 M elements): one mini-batch of N=8 folds + apply with the multi-tensor
    calls against one call per tensor.  GPU time by CUDA events, host time by perf_counter."""
    import paper_2305_19982_b200 as adama
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    sizes = []
    for _ in range(wl.CONFIG4_BLOCKS):
        sizes += [1600, 1600, 4800, 1600, 1600, 1600, 6400, 1600]
    sizes += [1600, 1600]
    N = wl.CONFIG4_N_MICRO
    ws = [wl.normal((n,), 0.02, torch.float32, 10 + i, device=dev) for i, n in enumerate(sizes)]
    ms = [torch.zeros(n, device=dev) for n in sizes]
    vs = [torch.zeros(n, device=dev) for n in sizes]
    gs = [wl.normal((n,), 1e-3, torch.bfloat16, 5000 + i, device=dev) for i, n in enumerate(sizes)]
    opt = adama.AdamA(wl.BETA1, wl.BETA2, wl.EPS, device=0)
    gl, ml, vl, wlst = (adama.TensorList(x) for x in (gs, ms, vs, ws))  # marshalled once
    res = {}
    for mode in ("multi", "per_tensor"):
        def step():
            opt.begin_minibatch(N)
            for _ in range(N):
                if mode == "multi":
                    opt.fold_multi(gl, ml, vl)
                else:
                    for g, m, v in zip(gs, ms, vs):
                        opt.fold(g, m, v)
            if mode == "multi":
                opt.apply_multi(wlst, ml, vl, wl.LR)
            else:
                for w, m, v in zip(ws, ms, vs):
                    opt.apply(w, m, v, wl.LR)
        for _ in range(3):
            step()
        torch.cuda.synchronize()
        l0 = opt.launch_count
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        host = (time.perf_counter() - t0) / args.steps
        torch.cuda.synchronize()
        res[mode] = {"gpu_ms_per_minibatch": e0.elapsed_time(e1) / args.steps,
                     "host_ms_per_minibatch": host * 1e3,
                     "launches_per_minibatch": (opt.launch_count - l0) // args.steps}
    print(json.dumps({"metric": "adama_small_tensor_minibatch_ms", "unit": "ms", "tensors": len(sizes),
                      "elements": sum(sizes), "n_micro": N, **res}), flush=True)
    opt.close()


def run_launch_check(args):
    """The multi-rank plumbing of the benchmark without any GPU work (used by the CPU tests with
    the gloo backend): rendezvous, barrier, a timed no-op region, max over ranks, one line."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group(args.backend)
        dist.barrier()
    t0 = time.perf_counter()
    time.sleep(0.01 * (rank + 1))
    t = torch.tensor([(time.perf_counter() - t0) * 1e3], dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"metric": "launch_check", "value": None, "n_gpus": world,
                          "ms_per_step": float(t.item()), "gpu_launches": 0,
                          "config": {"workload": "launch_check", "backend": args.backend}}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def relaunch_with_ranks(args):
    """`python bench.py --gpus N` started without a launcher: start the N ranks here, one per
    GPU, the way torchrun would (rendezvous on 127.0.0.1), and hand on their exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    # NCCL's communicator log (rings/trees, NVLS availability) goes to stderr with the run
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
           f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1", "--master-port", str(port),
           str(Path(__file__).resolve())] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--biases", action="store_true",
                    help="gpt2xl workload: give every linear layer a bias, folded in the fused launch")
    ap.add_argument("--flat-params", type=int, default=wl.CONFIG2_FULL_N)
    ap.add_argument("--linear-tokens", type=int, default=wl.CONFIG3.tokens,
                    help="tokens per micro-batch of the linear layer (default: the workload's 4096; "
                         "smaller values are for profiling the short-call kernel instance)")
    ap.add_argument("--linear-dims", type=int, nargs=2, default=None, metavar=("D_IN", "D_OUT"),
                    help="headline phase B on another layer shape (profiling runs; default 4096 4096)")
    ap.add_argument("--workload", default="headline", choices=["headline", "gpt2xl", "llama7b", "sweep", "small_tensors", "extensions", "oracle_timing", "wgrad_shapes", "launch_check"])
    ap.add_argument("--exchange", default="none", choices=["none", "allreduce", "sharded"],
                    help="N > 1: what the ranks exchange at the end of each mini-batch, inside the "
                         "timed step (none = independent replicas; allreduce = Section 3.3's state "
                         "all-reduce; sharded = reduce-scatter of the states, all-gather of the weights)")
    ap.add_argument("--backend", default="gloo", help="launch_check only: process-group backend")
    ap.add_argument("--layers-per-launch", type=int, default=1,
                    help="gpt2xl / llama7b workloads: consecutive layers folded by one grouped launch "
                         "(1 = one call per layer; 4 / 7 = one call per transformer block)")
    ap.add_argument("--stack-blocks", type=int, default=None,
                    help="gpt2xl / llama7b workloads: a shorter stack of that many blocks (profiling runs; "
                         "default: the workload's 48 / 32)")
    ap.add_argument("--stack-micro", type=int, default=None,
                    help="gpt2xl / llama7b workloads: micro-batches per mini-batch (profiling runs; "
                         "default: the workload's 8 / 16)")
    ap.add_argument("--inputs-settled", action="store_true",
                    help="gpt2xl / llama7b workloads: create the context with ADAMA_INPUTS_SETTLED")
    ap.add_argument("--no-stacks", action="store_true",
                    help="skip the two layer-stack workloads of the default line (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if (args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours"
            and args.workload in ("headline", "launch_check")):
        sys.exit(relaunch_with_ranks(args))
    if args.workload == "launch_check":
        run_launch_check(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.workload == "sweep":
        run_sweep(args)
    elif args.workload == "extensions":
        run_extensions(args)
    elif args.workload == "oracle_timing":
        run_oracle_timing(args)
    elif args.workload == "wgrad_shapes":
        run_wgrad_shapes(args)
    elif args.workload == "small_tensors":
        args.steps = min(args.steps, 10)
        run_small_tensors(args)
    elif args.workload != "headline":
        args.steps = min(args.steps, 3)
        run_stack(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
