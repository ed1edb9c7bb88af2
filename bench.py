#!/usr/bin/env python
"""Benchmark of one TwIST training round (BLOCKWISE) through the C ABI on B200.

A "step" is one whole round of the hot path over one batch of synthetic input:
sample masks -> per layer { gather -> K local steps (FFN block, QKV projection, output
projection: forward, MSE, backward with fused SGD; all S subnets per launch) -> aggregate }.
Metric: tokens/s per round, tokens = S * K * T.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead (a bounded
sample per step, extrapolated to a round; rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "twist_round_tokens_per_s"
UNIT = "tokens/s"
# Nominal peaks of the part (dense bf16 tensor throughput, HBM3e bandwidth); fractions against them are reported
# beside the fractions against the peaks measured on the machine.
# dram bytes (read + write) of one 7B-shaped gather launch from the committed ncu capture (profiles/)
NCU_GATHER_TRAFFIC = 1.42e9
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# algorithmic work of one round (what the method must do; the dense model would need more)
# ------------------------------------------------------------------------------------------------

def round_work(w, nq_valid=None):
    """FLOPs of the grouped GEMMs and bytes of gather / aggregate for one round."""
    S, K, T, d, L = w.n_subnets, w.local_steps, w.tokens, w.d_model, w.n_layers
    f = w.f_sub
    flops_ffn = 6.0 * T * d * f * w.nmat                      # fwd 2 + bwd 4 per weight element per token
    a = w.a_sub
    kv = (min(w.n_kv_heads, w.head_keep) * w.d_head) if w.n_heads else 0
    nq = (a + 2 * kv) if nq_valid is None else nq_valid
    flops_attn = 6.0 * T * d * (nq + a) if w.n_heads else 0.0
    gemm_flops = (flops_ffn + flops_attn) * S * K * L
    kept = (w.nmat * f + (nq + a if w.n_heads else 0)) * d    # kept elements per subnet per layer
    # read bf16, write bf16: the fp32 masters are not written by the gather, the first weight update of the round
    # creates them from the bf16 slice (that update then reads 2 instead of 4 bytes per element)
    gather_bytes = (2 + 2) * kept * S * L
    # aggregate: read every subnet's master (4 B) + write fp32 result and bf16 shadow for every covered element
    full = (w.nmat * w.d_ff + ((w.n_heads + 2 * w.n_kv_heads + w.n_heads) * w.d_head if w.n_heads else 0)) * d
    agg_bytes = 4 * kept * S * L + (4 + 2) * full * L         # cover mode: every element is covered
    return {"gemm_flops": gemm_flops, "gather_bytes": gather_bytes, "aggregate_bytes": agg_bytes, "full_elems": full}


# ------------------------------------------------------------------------------------------------
# N > 1: independent replicas, one process per GPU (the path has no exchange step between GPUs).
# ------------------------------------------------------------------------------------------------

def spawn_replicas(n: int, argv, extra_env=None, timeout=None) -> int:
    """Starts n copies of the command `argv`, one per GPU, with the environment a distributed launcher would give
    them (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, a free MASTER_PORT).  Rank 0's standard output
    passes through (it prints the one JSON line); the others' is dropped.  Returns the largest exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), **(extra_env or {}))
        procs.append(subprocess.Popen(argv, env=env, stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    for p in procs:
        try:
            rc = max(rc, abs(p.wait(timeout=timeout)))
        except subprocess.TimeoutExpired:
            p.kill()                       # the exact process this function started
            rc = max(rc, 124)
    return rc


def replica_seed(base: int, rank: int) -> int:
    """Every replica draws its own weights and batches."""
    return base + 7919 * rank


def max_over_ranks(ms_local: float, device="cuda") -> float:
    """Step time of the job = the slowest replica's (all-reduce MAX when a process group is up)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def whole_job_value(tokens_per_round: int, world: int, ms_per_step: float) -> float:
    """Tokens per second of all replicas together."""
    return world * tokens_per_round / (ms_per_step / 1e3)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()          # the exact process this object started
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm = sorted(float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit())
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) >= 9:
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (reported baseline and `--impl reference` arm)
# ------------------------------------------------------------------------------------------------

def oracle_round_estimate(w, tokens_sample=128, seed=7):
    """Times the oracle, as it stands, on a bounded sample of the workload: ONE layer, all S
    subnets, ONE local step on `tokens_sample` tokens per subnet, plus that layer's blueprint,
    gather and aggregate at full size.  The per-round figure scales the local-step time by
    K * T / tokens_sample and everything by the layer count (extrapolated)."""
    import numpy as np
    from dataclasses import replace
    from oracle import twist_oracle as o
    from paper_2511_03983_b200 import inputs as I

    lowp = w.dtype == I.DTYPE_BF16
    ws = replace(w, n_layers=1, local_steps=1, tokens=tokens_sample)
    mats = {"gate": I.MAT_GATE, "up": I.MAT_UP, "down": I.MAT_DOWN, "qkv": I.MAT_QKV, "o": I.MAT_O}
    names = ["up", "down"] + (["gate"] if w.ffn_kind == I.FFN_SWIGLU else []) + (["qkv", "o"] if w.n_heads else [])
    full = {m: I.weight(ws, 0, mats[m]).astype(np.float64) for m in names}
    cache = {}

    def get_batch(kind, rnd, s, k, width):
        key = (kind, s, width)
        if key not in cache:
            cache[key] = I.batch(ws, kind, rnd, s, k, width).astype(np.float64)
        return cache[key]

    t0 = time.perf_counter()
    bp = o.layer_blueprints(ws, 0, 0)
    t1 = time.perf_counter()
    slices = [{m: np.asarray(v, dtype=np.float64) for m, v in o.gather_layer(ws, full, bp, s).items()}
              for s in range(ws.n_subnets)]
    t2 = time.perf_counter()
    for s in range(ws.n_subnets):     # warm the batch cache outside the timed local steps
        get_batch(0, 0, s, 0, w.d_model), get_batch(1, 0, s, 0, w.d_model)
        if w.n_heads:
            get_batch(2, 0, s, 0, slices[s]["qkv"].shape[0]), get_batch(3, 0, s, 0, slices[s]["o"].shape[0])
    t3 = time.perf_counter()
    for s in range(ws.n_subnets):
        o.local_steps_blockwise(ws, slices[s], get_batch, 0, s, lowp)
    t4 = time.perf_counter()
    o.aggregate_layer(ws, full, slices, bp)
    t5 = time.perf_counter()
    t_mask, t_gather, t_local, t_agg = t1 - t0, t2 - t1, t4 - t3, t5 - t4
    per_round = w.n_layers * (t_mask + t_gather + t_agg + t_local * w.local_steps * (w.tokens / tokens_sample))
    cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        pass
    return {
        "value": w.tokens_per_round / per_round, "unit": UNIT, "cores": cores, "kind": "oracle",
        "sample": (f"1 of {w.n_layers} layers, all S={w.n_subnets} subnets, 1 local step on {tokens_sample} of "
                   f"{w.tokens} tokens per subnet (numpy fp64), blueprint+gather+aggregate of that layer at full "
                   f"size; extrapolated to a round: layers x (mask {t_mask:.3f}s + gather {t_gather:.3f}s + aggregate "
                   f"{t_agg:.3f}s + local {t_local:.3f}s x K x T/{tokens_sample})"),
        "sample_seconds": round(t5 - t0, 3), "round_seconds_extrapolated": round(per_round, 1),
    }


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times, last = [], None
    for i in range(args.warmup + args.steps):
        last = oracle_round_estimate(w, tokens_sample=args.oracle_tokens)
        if i >= args.warmup:
            times.append(last["round_seconds_extrapolated"])
    ms = 1e3 * sum(times) / len(times)
    value = w.tokens_per_round / (ms / 1e3)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": workload_config(w, args),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_config(w, args):
    if getattr(args, "mode", "blockwise") == "stack":
        return {"workload": f"configs[{args.config - 1}] {w.name}: STACK round (chained layers, causal attention core, "
                            f"{w.n_seqs} sequences of {w.tokens // w.n_seqs}), L={w.n_layers} d={w.d_model} F={w.d_ff} "
                            f"f'={w.f_sub} H'={w.head_keep}/{w.n_heads} S={w.n_subnets} T={w.tokens} K={w.local_steps}",
                "tokens_per_round": w.tokens_per_round, "mode": "stack, all layers resident",
                "l2_policy": "working set exceeds L2 across the layers of a round",
                "parallelism": "replicas only" if args.gpus > 1 else "single GPU"}
    hybrid = getattr(args, "mode", "blockwise") == "hybrid"
    masked = getattr(args, "mode", "blockwise") == "masked"
    sharded = getattr(args, "mode", "blockwise") == "sharded"
    return {"workload": f"configs[{args.config - 1}] {w.name}: {'HYBRID ' if hybrid else 'MASKED ' if masked else ''}BLOCKWISE round, L={w.n_layers} d={w.d_model} "
                        f"F={w.d_ff} f'={w.f_sub} H'={w.head_keep}/{w.n_heads} S={w.n_subnets} T={w.tokens} K={w.local_steps}",
            "tokens_per_round": w.tokens_per_round,
            "mode": ("hybrid: worker 0 masked on the full-width model in place, the others on gathered slices; flops "
                     "counted are those of the gathered subnets" if hybrid else
                     "masked: every worker a full-width copy under its activation mask; flops counted are those of the "
                     "gathered subnets" if masked else
                     "blockwise, layers streamed; the S subnets of one round spread over the GPUs, aggregate = partial "
                     "sums + all-reduce + division" if sharded else "blockwise, layers streamed"),
            "l2_policy": "inputs larger than L2 (every tensor a kernel reads is >= 4x the 126 MB L2)"
                         if w.d_model >= 2048 else "working set exceeds L2 across the layers of a round",
            "parallelism": (f"subnets sharded over {args.gpus} GPUs" if sharded and args.gpus > 1 else
                            "replicas only" if args.gpus > 1 else "single GPU")}


# ------------------------------------------------------------------------------------------------
# CUDA arm
# ------------------------------------------------------------------------------------------------

def run_ours(args, w):
    import torch
    import torch.distributed as dist

    from paper_2511_03983_b200 import binding as B
    from paper_2511_03983_b200 import inputs as I
    from paper_2511_03983_b200.engine import (HybridRoundEngine, MaskedRoundEngine, RoundEngine, ShardedRoundEngine,
                                              StackEngine)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B.lib()
    bf16 = w.dtype == I.DTYPE_BF16
    td = torch.bfloat16 if bf16 else torch.float32
    stack = args.mode == "stack"
    if stack:
        if not (w.n_heads and bf16 and w.tokens % w.n_seqs == 0):
            raise SystemExit("--mode stack needs a bf16 workload with attention heads")
        eng = StackEngine(w, w.n_seqs, w.tokens // w.n_seqs, keep_f32_full=True)
    elif args.mode in ("hybrid", "masked"):
        if w.n_heads or not bf16:
            raise SystemExit(f"--mode {args.mode} needs a bf16 FFN-only workload (--config 5)")
        if args.mode == "hybrid":
            eng = HybridRoundEngine(w, compute_dx=True, fuse_loss=True, store_outputs=False)
        else:
            eng = MaskedRoundEngine(w, keep_f32_full=True, compute_dx=True, fuse_loss=True, store_outputs=False)
    elif args.mode == "sharded":                          # the S subnets of ONE round spread over the GPUs
        eng = ShardedRoundEngine(w, rank=rank, world=world, keep_f32_full=True, compute_dx=True, fuse_loss=True,
                                 store_outputs=False)
    else:
        eng = RoundEngine(w, keep_f32_full=True, compute_dx=True, fuse_loss=True, store_outputs=False)
    sharded = args.mode == "sharded"
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed_w if sharded else replica_seed(w.seed_w, rank))      # sharded: one model on every GPU
    for m, v in eng.full.items():                         # weights ~ N(0, 0.02^2), one matrix at a time
        for l in range(w.n_layers):
            v[l].copy_((torch.randn(v[l].shape, generator=gen, device="cuda", dtype=torch.float32) * 0.02).to(td))
            if args.mode == "hybrid":                     # the central worker trains on the fp32 full model in place
                eng.full_f32[m][l].copy_(v[l])
    gen.manual_seed(replica_seed(w.seed_x, rank))
    S, T, K = eng.w.n_subnets, w.tokens, w.local_steps     # (sharded: this GPU's subnets)
    widths = [("X", w.d_model), ("Td", w.d_model)] + ([("Tq", eng.nq), ("A", eng.a_sub)]
                                                      if (eng.has_attn and not stack) else [])
    host = {}
    for name, width in widths:
        lst = getattr(eng, name)
        for k in range(K):
            t = torch.empty(S, T, width, dtype=td, device="cuda")
            for s in range(S):
                t[s].copy_(torch.randn(T, width, generator=gen, device="cuda", dtype=torch.float32).to(td))
            lst.append(t)
    h2d_bytes = sum(t.numel() * t.element_size() for name, _ in widths for t in getattr(eng, name))
    loss_dev = eng.stack_loss if stack else eng.loss
    d2h_bytes = loss_dev.numel() * 4

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing -------------------------------------------------------------
    rnd = 0
    for _ in range(args.warmup):
        eng.run_round(rnd)
        rnd += 1
    barrier()
    eng.launches = 0
    eng.timing = True
    eng.events.clear()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        eng.run_round(rnd)
        rnd += 1
    e1.record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = e0.elapsed_time(e1)
    launches = eng.launches
    phases = eng.phase_ms()
    eng.timing = False
    status = B.twist_device_status()
    if status != 0:
        raise SystemExit(f"device status {status}: a bounded device wait expired")
    ms_per_step = max_over_ranks(ms_total) / args.steps
    # replicas: every GPU runs a whole round of its own; sharded: all GPUs together run one round
    job_world = 1 if sharded else world
    value = whole_job_value(w.tokens_per_round, job_world, ms_per_step)

    # ---- end-to-end: host buffers, copies inside the timed region --------------------------------
    e2e = None
    if not args.no_e2e:
        # Host side of the copies.  One replica pins all K batches of a round (distinct data per local step).  With
        # several replicas on one host that would pin N x 25.8 GB, so each then pins one local step's batches and
        # copies them K times per round: the same bytes cross the bus, the host memory stays bounded.
        pinned = {}
        for name, _ in widths:
            lst = getattr(eng, name)
            if world == 1:
                pinned[name] = [t.cpu().pin_memory() for t in lst]
            else:
                one = lst[0].cpu().pin_memory()
                pinned[name] = [one] * len(lst)
        loss_host = torch.empty(loss_dev.shape, dtype=torch.float32).pin_memory()
        n_e2e = max(1, min(args.steps, args.e2e_steps))
        # Two sets of device batch buffers: while a round runs on one, the next step's batches are copied into
        # the other on a second stream (what a training loop's data prefetcher does).  Step 0's copy is exposed.
        sets = [{name: getattr(eng, name) for name, _ in widths},
                {name: [torch.empty_like(t) for t in getattr(eng, name)] for name, _ in widths}]
        copy_stream = torch.cuda.Stream()
        main = torch.cuda.current_stream()
        copied = [torch.cuda.Event() for _ in range(n_e2e)]
        done = [torch.cuda.Event() for _ in range(n_e2e)]

        def issue_copy(i):
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(done[i - 2])          # the round that last read this buffer set
                for name, _ in widths:
                    for dst, src in zip(sets[i % 2][name], pinned[name]):
                        dst.copy_(src, non_blocking=True)
                copied[i].record(copy_stream)

        barrier()
        e0.record()
        copy_stream.wait_event(e0)
        issue_copy(0)
        for i in range(n_e2e):
            if i + 1 < n_e2e:
                issue_copy(i + 1)
            main.wait_event(copied[i])
            for name, _ in widths:
                setattr(eng, name, sets[i % 2][name])
            eng.run_round(rnd)
            rnd += 1
            done[i].record(main)
            loss_host.copy_(loss_dev, non_blocking=True)
        e1.record()
        barrier()
        for name, _ in widths:
            setattr(eng, name, sets[0][name])
        e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / n_e2e
        e2e = {"value": whole_job_value(w.tokens_per_round, job_world, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": d2h_bytes, "steps": n_e2e,
               "note": "pinned host batches copied in (the next step's copy overlaps the current round on a second "
                       "stream), per-subnet losses copied out, every step"
                       + ("" if world == 1 else "; each replica pins one local step's batches and copies them K times")}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    work = round_work(eng.w if sharded else w)            # per GPU (sharded: its S / N subnets)
    if sharded:     # the aggregate in two halves: sums of the GPU's subnets written for the whole layer (4 B per element),
        full = work.pop("full_elems")     # then the reduced sums read and the fp32 model + bf16 shadow written (4 + 4 + 2)
        work["aggregate_bytes"] += (4 + 4) * full * w.n_layers
    else:
        work.pop("full_elems")
    if args.mode == "hybrid":                             # worker 0 has no slice: S - 1 subnets are gathered
        work["gather_bytes"] *= (w.n_subnets - 1) / w.n_subnets
    if args.mode == "masked":                             # every worker copies and returns the whole layer
        full_over_kept = w.n_ffn_blocks / w.ffn_keep
        work["gather_bytes"] *= full_over_kept            # (the aggregate reads the same rows as in the gathered round)
    gemm_names = [n for n in ("ffn_fwd", "ffn_bwd", "qkv_fwd", "qkv_bwd", "o_fwd", "o_bwd") if n in phases]
    gemm_ms = sum(phases[n][0] for n in gemm_names)
    gemm_launches_per_round = w.n_layers * K * ((2 + 4) + ((1 + 2 + 1 + 2) if eng.has_attn else 0))
    roofline, phase_out = None, {}
    for n, (ms, calls) in phases.items():
        phase_out[n] = {"ms_per_step": ms / args.steps, "calls_per_step": calls // args.steps}
    if bf16 and gemm_ms > 0:
        tflops = work["gemm_flops"] * args.steps / (gemm_ms / 1e3) / 1e12
        # Denominator: the sustained cuBLAS figure when the step ran power-capped (the 7B-shaped rounds), the burst
        # figure when the SM clock stayed at its maximum (short launches between lighter kernels).
        capped = bool(clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz")
                      and clocks["sm_mhz"] < 0.95 * clocks["sm_max_mhz"])
        peak_key = "bf16_tflops_sustained" if capped or not clocks or not clocks.get("sm_mhz") else "bf16_tflops"
        peak = peaks[peak_key]
        roofline = {"bound": "tensor", "kernel": "gemm_kernel (grouped tcgen05 GEMM, all layouts/epilogues)",
                    "achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak,
                    "peak_source": f"{peak_key} of {peaks['source']}",
                    "frac_of_nominal": tflops / NOMINAL_BF16_TFLOPS, "nominal_peak": NOMINAL_BF16_TFLOPS,
                    # what the same kernels would give at the maximum SM clock, if throughput followed the clock
                    # (the step runs under the power cap): achieved x max MHz / median MHz
                    "achieved_at_max_clock": (tflops * clocks["sm_max_mhz"] / clocks["sm_mhz"]
                                              if clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") else None),
                    # dram read + write bytes per launch: the counters on file (profiles/) were taken at this size
                    # before the kernel's tiles were synchronised; the kernel has changed since, so: null
                    "traffic": None,
                    "flops_per_launch": work["gemm_flops"] / gemm_launches_per_round,
                    "avg_launch_ms": gemm_ms / args.steps / gemm_launches_per_round,
                    "share_of_step": gemm_ms / ms_total}
    hbm = {}
    # DRAM bytes per launch from the committed ncu capture of one 7B-shaped layer (profiles/); only that launch shape
    ncu_traffic = {"gather": NCU_GATHER_TRAFFIC, "aggregate": 2.79e9} if (args.config == 4 and not stack) else {}
    for name, key in (("gather", "gather_bytes"), ("aggregate", "aggregate_bytes")):
        if name in phases and phases[name][0] > 0:
            gbs = work[key] * args.steps / (phases[name][0] / 1e3) / 1e9
            hbm[name] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal": gbs / NOMINAL_HBM_GBS,
                         "nominal_peak": NOMINAL_HBM_GBS, "bytes_per_launch": work[key] / w.n_layers,
                         "traffic": ncu_traffic.get(name)}
    if roofline is None and "aggregate" in hbm:
        roofline = dict(hbm["aggregate"], kernel="aggregate_rows_kernel")

    cpu = None
    if not args.no_cpu_baseline:
        cpu = oracle_round_estimate(w, tokens_sample=args.oracle_tokens)
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if sharded else "weak",
           "vs_baseline": None,
           "dtype": "bf16" if bf16 else "f32", "data": "synthetic", "config": workload_config(w, args),
           "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "hbm_kernels": hbm,
           "phases": phase_out, "cpu_baseline": cpu}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Workload 5: the gather / aggregate sweep over S x keep on the 7B FFN shapes (IID masks, K=1, 1024 tokens per
    subnet).  One JSON line whose `cells` give the gather and scatter-average GB/s of every cell."""
    import torch
    from dataclasses import replace
    from paper_2511_03983_b200 import binding as B
    from paper_2511_03983_b200 import inputs as I
    from paper_2511_03983_b200.engine import RoundEngine

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    B.lib()
    peaks = measured_peaks()
    cells = []
    for w in I.sweep_cfg5():
        if args.layers:
            w = replace(w, n_layers=args.layers)
        eng = RoundEngine(w, keep_f32_full=True, compute_dx=True, fuse_loss=True, store_outputs=False)
        gen = torch.Generator(device="cuda")
        gen.manual_seed(w.seed_w)
        for m, v in eng.full.items():
            for l in range(w.n_layers):
                v[l].copy_((torch.randn(v[l].shape, generator=gen, device="cuda", dtype=torch.float32) * 0.02).to(v.dtype))
        for name in ("X", "Td"):
            getattr(eng, name).append(torch.randn(w.n_subnets, w.tokens, w.d_model, generator=gen, device="cuda",
                                                  dtype=torch.float32).to(torch.bfloat16))
        for r in range(max(1, args.warmup)):
            eng.run_round(r)
        torch.cuda.synchronize()
        eng.timing = True
        eng.events.clear()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for r in range(args.steps):
            eng.run_round(100 + r)
        e1.record()
        torch.cuda.synchronize()
        ph = eng.phase_ms()
        if B.twist_device_status() != 0:
            raise SystemExit("device status: a bounded device wait expired")
        kept = w.nmat * w.f_sub * w.d_model                                      # kept elements per subnet and layer
        covered = int((eng.cover_ffn != 0).sum().item()) * w.ffn_block * w.d_model * w.nmat   # last round, all layers
        gather_b = 4.0 * kept * w.n_subnets * w.n_layers
        agg_b = 4.0 * kept * w.n_subnets * w.n_layers + 6.0 * covered
        g_gbs = gather_b * args.steps / (ph["gather"][0] / 1e3) / 1e9
        a_gbs = agg_b * args.steps / (ph["aggregate"][0] / 1e3) / 1e9
        cells.append({"S": w.n_subnets, "keep": round(w.ffn_keep / w.n_ffn_blocks, 2), "gather_gbs": round(g_gbs, 1),
                      "aggregate_gbs": round(a_gbs, 1), "gather_frac": round(g_gbs / peaks["hbm_gbs"], 3),
                      "aggregate_frac": round(a_gbs / peaks["hbm_gbs"], 3),
                      "covered_fraction": round(covered / (w.nmat * w.d_ff * w.d_model * w.n_layers), 4),
                      "round_ms": round(e0.elapsed_time(e1) / args.steps, 2),
                      "tokens_per_s": round(w.tokens_per_round / (e0.elapsed_time(e1) / args.steps / 1e3), 1)})
        del eng
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "gather_and_aggregate_gbs", "unit": "GB/s", "peak": peaks["hbm_gbs"],
                      "peak_source": f"hbm_gbs of {peaks['source']}", "steps": args.steps, "warmup": max(1, args.warmup),
                      "config": {"workload": "configs[4] gather/aggregate sweep on the 7B FFN shapes: d=4096 F=11008 "
                                             f"L={args.layers or 32} bf16 weights, fp32 aggregate, IID masks, K=1, "
                                             "1024 tokens per subnet",
                                 "bytes": "gather 4 B per kept element (2 read, 2 write; the fp32 masters are created by "
                                          "the first weight update); aggregate 4 B per kept master element + 6 B per "
                                          "covered element"},
                      "cells": cells}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=4, help="workload 1..5 (default 4: the 7B-shaped round)")
    ap.add_argument("--oracle-tokens", type=int, default=128)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling on a small case)")
    ap.add_argument("--tokens", type=int, default=0, help="override tokens per subnet-step (profiling on a small case)")
    ap.add_argument("--local-steps", type=int, default=0)
    ap.add_argument("--mode", default="blockwise", choices=["blockwise", "stack", "hybrid", "masked", "sharded"],
                    help="stack: chained layers with the attention core (workloads 2 and 3); hybrid: worker 0 trains "
                         "the full-width model under a mask; masked: every worker does (FFN-only workload 5)")
    ap.add_argument("--sweep", action="store_true", help="workload 5: all 12 (S, keep) cells, gather / aggregate GB/s")
    args = ap.parse_args()
    from dataclasses import replace
    from paper_2511_03983_b200 import inputs as I
    w = I.PRESETS[args.config]
    if args.layers:
        w = replace(w, n_layers=args.layers, name=w.name + f"-L{args.layers}")
    if args.tokens:
        w = replace(w, tokens=args.tokens, name=w.name + f"-T{args.tokens}")
    if args.local_steps:
        w = replace(w, local_steps=args.local_steps, name=w.name + f"-K{args.local_steps}")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not args.sweep:
        # started as a plain command: become the launcher of one replica per GPU (replicas only, no collective)
        raise SystemExit(spawn_replicas(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args, w)
    elif args.sweep:
        run_sweep(args)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
