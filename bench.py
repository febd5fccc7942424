#!/usr/bin/env python
"""Benchmark of the KV-cache compression path on B200.

A step is one kvm_compress call (score -> segment -> pivot -> merge+compact) over
one Llama2-7B-shaped attention layer: batch 1, 32 heads, head_dim 128, 4096
tokens, bf16, 50 % budget.  Inputs are seeded synthetic tensors; several layers'
worth of inputs are rotated so that each step reads tensors that are not in L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

The timed region is K steps between two CUDA events; it is repeated until at least
half a second of GPU time has been measured, and the line reports the mean, the
median and the best block.  Prints one JSON line (rank 0).  With --gpus N > 1 and no
torchrun environment the script starts the N ranks itself.  `--impl reference` times
the fp64 CPU checker on the host cores instead (a deliberately plain program,
reported for context).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2407_08454_b200 import replicas
from paper_2407_08454_b200 import synth_inputs as si

WORKLOAD = "C1"
METRIC = "KV tokens compressed/s (all layers, heads)"
UNIT = "KV tokens/s"
N_BUFFERS = 3  # rotating input sets: 3 x 100 MB > 126 MB of L2
MIN_TIMED_MS = 500.0  # the timed block is repeated until this much GPU time has been measured
# dram__bytes_read.sum + dram__bytes_write.sum of one column-pass launch on this workload, from the ncu capture
# summarised in profiles/score_tc_column_pass_C1.md (None when the kernel has changed since that capture)
NCU_TRAFFIC_BYTES_COLUMN_PASS = 71.38e6 + 3.14e6
OTHER_WORKLOADS = ("C2", "C3", "C4")
LAYERS_PER_WORKLOAD = 3


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _names(self, mask: int):
        nv = self.nv
        table = [("sw_power_cap", "nvmlClocksThrottleReasonSwPowerCap"),
                 ("hw_slowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("sw_thermal_slowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("hw_power_brake", "nvmlClocksThrottleReasonHwPowerBrakeSlowdown"),
                 ("sync_boost", "nvmlClocksThrottleReasonSyncBoost"),
                 ("applications_clocks", "nvmlClocksThrottleReasonApplicationsClocksSetting")]
        return [n for n, attr in table if hasattr(nv, attr) and (mask & getattr(nv, attr))]

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.reasons.update(self._names(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)))
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def algorithmic_work(cfg):
    """Per-layer work the method must do (causal half of QK^T only; K and V read once per consumer)."""
    B, Hq, Hkv, S, D = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim
    e = 2 if cfg.dtype == "bf16" else 4
    flops_pass = 2.0 * D * (S * (S + 1) / 2.0) * Hq * B
    kv = B * Hkv * S * D * e
    return {"flops_per_score_pass": flops_pass, "k_bytes": kv, "q_bytes": B * Hq * S * D * e}


# ----------------------------------------------------------------------------- input generation on a process pool
def _gen_heads(args):
    """Worker: a few KV heads (and their query groups) of one layer, as raw int16/float32 arrays."""
    name, layer, heads = args
    cfg = si.CONFIGS[name]
    d = si.make_layer(cfg, layer, kv_heads=heads)
    view = torch.int16 if cfg.dtype == "bf16" else torch.float32
    return heads, {k: v.view(view).numpy() for k, v in d.items()}


def generate_layers(pool, name: str, layers):
    """The layers of workload `name`, generated head by head on the pool (every head has its own random stream, so
    the result equals si.make_layer of the whole layer).  Returns a list of {"Q","K","V"} CPU tensors."""
    cfg = si.CONFIGS[name]
    jobs = [(name, l, [h]) for l in layers for h in range(cfg.n_kv_heads)]
    parts = pool.map(_gen_heads, jobs, chunksize=1)
    out = []
    G = cfg.group
    per_layer = cfg.n_kv_heads
    for li, _ in enumerate(layers):
        chunk = parts[li * per_layer:(li + 1) * per_layer]
        tens = {}
        for key, heads_mult in (("Q", G), ("K", 1), ("V", 1)):
            arr = np.concatenate([c[1][key] for c in chunk], axis=1)
            t = torch.from_numpy(arr)
            tens[key] = t.view(cfg.torch_dtype) if cfg.dtype == "bf16" else t
        out.append(tens)
    return out


# ----------------------------------------------------------------------------- the CPU checker's arm
def run_reference(args, cfg):
    """The fp64 CPU checker as it stands, on a bounded sample of the workload per step."""
    from oracle import kvmo
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    units_per_step = 4
    d = si.make_layer(cfg, 0, kv_heads=list(range(units_per_step)))
    def step():
        kvmo.compress(d["Q"], d["K"], d["V"], float(np.float32(cfg.budget)), float(np.float32(0.17)),
                      float(np.float32(0.12)))
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = args.steps * units_per_step * cfg.seq / dt
    sample = f"{units_per_step} of {cfg.n_kv_heads} units of one {WORKLOAD} layer per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": cfg.batch, "heads": cfg.n_q_heads, "seq_len": cfg.seq,
                   "head_dim": cfg.head_dim, "budget": cfg.budget, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": kvmo.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def spawn_ranks(n: int) -> int:
    """Started without a torchrun environment and asked for several GPUs: start one rank per GPU ourselves."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def stats_of(ms_list):
    a = np.asarray(ms_list, dtype=np.float64)
    return {"mean": float(a.mean()), "median": float(np.median(a)), "best": float(a.min()), "n": int(a.size)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="skip the C2-C4 section of extras")
    ap.add_argument("--min-ms", type=float, default=MIN_TIMED_MS,
                    help="GPU time to accumulate over repeated timed blocks (profiler captures use a small value)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = si.CONFIGS[WORKLOAD]
    if args.impl == "reference":
        return run_reference(args, cfg)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    solo = rank == 0 and world == 1
    # The pool that generates inputs (and nothing else) is started before the first CUDA call.
    pool = None
    if solo and not args.no_workloads:
        import multiprocessing as mp
        pool = mp.get_context("spawn").Pool(min(16, os.cpu_count() or 1))

    import paper_2407_08454_b200 as kvm
    from paper_2407_08454_b200 import build as kbuild
    kbuild.build()

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    # ---- inputs: N_BUFFERS distinct layers per rank (weak scaling: every rank compresses its own layers)
    p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype,
                        budget=cfg.budget)
    host = [si.make_layer(cfg, layer=l) for l in replicas.layers_for_rank(rank, world, N_BUFFERS)]
    bufs = [{k: v.to(dev) for k, v in h.items()} for h in host]
    comp = kvm.Compressor(p, device=dev)
    stats = kvm.new_stats(dev)
    U = cfg.batch * cfg.n_kv_heads
    kv_tokens_per_step = U * cfg.seq
    stream = torch.cuda.current_stream()
    n_calls = 0

    def step(i, rotate=True):
        b = bufs[i % N_BUFFERS if rotate else 0]
        kvm.kvm_compress(p, b["Q"], b["K"], b["V"], comp.K_out, comp.V_out, comp.out_len, comp.out_pos, None, stats,
                         comp.ws, stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_blocks(fn, steps, min_ms=args.min_ms, max_blocks=400):
        """Blocks of `steps` calls between two events each, repeated until min_ms of GPU time; every rank runs the
        same number of blocks (the count is fixed from the first block's slowest-rank time)."""
        def one_block():
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            e0.record(stream)
            for i in range(steps):
                fn(i)
            e1.record(stream)
            barrier()
            return replicas.slowest_rank_ms(e0.elapsed_time(e1), dist, dev)
        first = one_block()
        blocks = int(min(max_blocks, max(1, math.ceil(min_ms / max(first, 1e-3)))))
        return [first] + [one_block() for _ in range(blocks - 1)]

    for i in range(args.warmup):
        step(i)
        n_calls += 1
    barrier()
    with ClockSampler(physical_gpu_index(local)) as clk:
        block_ms = timed_blocks(step, args.steps)
    n_calls += len(block_ms) * args.steps
    per_step = stats_of([b / args.steps for b in block_ms])
    ms_per_step = sum(block_ms) / (len(block_ms) * args.steps)
    value = replicas.aggregate_throughput(world, args.steps, kv_tokens_per_step, ms_per_step * args.steps)
    st = kvm.read_stats(stats)
    assert st.status == 0, "device reported an error status"
    # the same step on one input set that stays in L2 between calls (the working set of a layer is of L2's size)
    warm_ms = timed_blocks(lambda i: step(i, rotate=False), args.steps, min_ms=min(100.0, args.min_ms))
    l2_warm = stats_of([b / args.steps for b in warm_ms])

    # ---- per-kernel timing (same launches, event pairs around each public step)
    b0 = bufs[0]
    scores = torch.empty(cfg.batch, cfg.n_kv_heads, cfg.seq, device=dev)
    lses = [torch.empty(cfg.batch, cfg.n_q_heads, cfg.seq, device=dev) for _ in range(N_BUFFERS)]
    set_start = torch.empty(cfg.batch, cfg.n_kv_heads, comp.cap + 1, dtype=torch.int32, device=dev)

    def timed(fn, reps):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(reps):
            fn(i)
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    reps = max(10, min(args.steps, 200))
    ws = comp.ws
    t_score = timed(lambda i: kvm.kvm_score(p, bufs[i % N_BUFFERS]["Q"], bufs[i % N_BUFFERS]["K"], None, scores, ws,
                                            stream), reps)
    # natural-log row log-sum-exp of every input set from the library's own row pass, so that the column pass
    # can be timed alone through the public lse_in argument, on rotating inputs like the rest
    for bi, lse_b in zip(bufs, lses):
        kvm.kvm_row_lse(p, bi["Q"], bi["K"], lse_b, ws, stream)
    t_rowpass = timed(lambda i: kvm.kvm_row_lse(p, bufs[i % N_BUFFERS]["Q"], bufs[i % N_BUFFERS]["K"],
                                                lses[i % N_BUFFERS], ws, stream), reps)
    t_colsum = timed(lambda i: kvm.kvm_score(p, bufs[i % N_BUFFERS]["Q"], bufs[i % N_BUFFERS]["K"],
                                             lses[i % N_BUFFERS], scores, ws, stream), reps)
    t_segment = timed(lambda i: kvm.kvm_segment(p, bufs[i % N_BUFFERS]["K"], scores, None, set_start, comp.out_pos,
                                                comp.out_len, None, None, ws, stream), reps)
    t_merge = timed(lambda i: kvm.kvm_merge_compact(p, bufs[i % N_BUFFERS]["K"], bufs[i % N_BUFFERS]["V"], set_start,
                                                    comp.out_pos, comp.out_len, comp.K_out, comp.V_out, None, ws,
                                                    stream), reps)
    work = algorithmic_work(cfg)
    peaks = measured_peaks()
    achieved = work["flops_per_score_pass"] / (t_colsum * 1e-3) / 1e12
    out_rows = int(comp.out_len.sum().item())
    merge_bytes = 2 * work["k_bytes"] + 2 * out_rows * cfg.head_dim * 2
    roofline = {
        "kernel": "score column pass (kvm_score with lse_in)", "bound": "tensor", "achieved": achieved,
        "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
        "traffic": NCU_TRAFFIC_BYTES_COLUMN_PASS,
        "algorithmic_bytes": work["q_bytes"] + work["k_bytes"] + cfg.batch * cfg.n_q_heads * cfg.seq * 32
                             + U * cfg.seq * 4,
        "peak_source": peaks["source"] + " burst bf16",
    }
    # the same kernel against the unit that actually limits it: one exponential per causal logit on the
    # special-function units (16 results per clock per SM)
    exps_per_pass = cfg.batch * cfg.n_q_heads * cfg.seq * (cfg.seq + 1) / 2.0
    sfu_peak = 16.0 * torch.cuda.get_device_properties(dev).multi_processor_count * (clk.max_mhz or 1965) * 1e6
    roofline_sfu = {
        "kernel": roofline["kernel"], "bound": "alu", "unit": "Gexp/s",
        "achieved": exps_per_pass / (t_colsum * 1e-3) / 1e9, "peak": sfu_peak / 1e9,
        "frac": exps_per_pass / (t_colsum * 1e-3) / sfu_peak,
        "peak_source": "16 ex2 per clock per SM x SM count x maximum SM clock",
    }
    kernels = {
        "score_both_passes_ms": t_score, "score_row_pass_ms": t_rowpass, "score_column_pass_ms": t_colsum,
        "similarity_segment_ms": t_segment, "merge_compact_ms": t_merge,
        "merge_compact_gbs": merge_bytes / (t_merge * 1e-3) / 1e9,
        "segment_gbs": (work["k_bytes"] + 3 * 4 * U * cfg.seq) / (t_segment * 1e-3) / 1e9,
        "score_both_passes_tflops": 2 * work["flops_per_score_pass"] / (t_score * 1e-3) / 1e12,
    }
    # fraction of each step's own roofline (measured peaks): tensor for the score passes, HBM for the rest
    kernels["roofline_frac"] = {
        "score_both_passes": kernels["score_both_passes_tflops"] / peaks["bf16_tflops"],
        "score_column_pass": achieved / peaks["bf16_tflops"],
        "similarity_segment": kernels["segment_gbs"] / peaks["hbm_gbs"],
        "merge_compact": kernels["merge_compact_gbs"] / peaks["hbm_gbs"],
    }
    # the target's denominator: slower of score flops at tensor peak and total bytes at HBM bandwidth
    total_bytes = work["q_bytes"] + 2 * work["k_bytes"] + 2 * out_rows * cfg.head_dim * 2
    t_roof_ms = max(2 * work["flops_per_score_pass"] / (peaks["bf16_tflops"] * 1e12),
                    total_bytes / (peaks["hbm_gbs"] * 1e9)) * 1e3
    e2e_frac = t_roof_ms / ms_per_step

    # ---- beyond the headline path, same workload: the method's variants, the ratio statistic and the
    # decode-step attention used for the output-perturbation check (each timed alone, CUDA events)
    def params(**rules):
        kw = dict(budget=cfg.budget)
        kw.update(rules)
        return kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype, **kw)

    def t_compress(pv, inputs=None, stats_buf=None):
        assert kvm.kvm_workspace_bytes(pv) <= ws.numel()
        src = inputs or bufs
        return timed(lambda i: kvm.kvm_compress(pv, src[i % len(src)]["Q"], src[i % len(src)]["K"],
                                                src[i % len(src)]["V"], comp.K_out, comp.V_out, comp.out_len,
                                                comp.out_pos, None, stats_buf, ws, stream), min(reps, 50))

    key = torch.rand(cfg.batch, cfg.n_kv_heads, cfg.seq, device=dev)
    p_anchor = params(set_rule=kvm.KVM_SETS_ANCHOR, enforce_budget=0)      # capacity S: its own buffers
    comp_a = kvm.Compressor(p_anchor, device=dev)
    t_anchor = timed(lambda i: kvm.kvm_compress(p_anchor, bufs[i % N_BUFFERS]["Q"], bufs[i % N_BUFFERS]["K"],
                                                bufs[i % N_BUFFERS]["V"], comp_a.K_out, comp_a.V_out, comp_a.out_len,
                                                comp_a.out_pos, None, None, comp_a.ws, stream), min(reps, 50))
    del comp_a
    extras = {
        "compress_anchor_sets_ms": t_anchor,
        "compress_average_last_pivot_ms": t_compress(params(pivot_rule=kvm.KVM_PIVOT_LAST,
                                                            weight_rule=kvm.KVM_WEIGHT_AVERAGE)),
        "compress_keyed_pivot_ms": t_compress(params(pivot_rule=kvm.KVM_PIVOT_KEY, pivot_key=key)),
        "compress_pivot_only_ms": t_compress(params(weight_rule=kvm.KVM_WEIGHT_PIVOT_ONLY)),
        "compress_set_sigma_ms": t_compress(params(weight_rule=kvm.KVM_WEIGHT_SET_SIGMA)),
        "compress_eviction_ms": t_compress(params(set_rule=kvm.KVM_SETS_CONSERVED_ONLY, recent_ratio=0.17,
                                                  heavy_ratio=cfg.budget - 0.17)),
    }
    # a case in which the budget rule fires: weakly correlated keys (rho 0.6: most neighbour pairs fall below
    # the threshold, so the sets outnumber the capacity) at the 35 % budget, same shape as the headline workload
    cfg_b = cfg.scaled(rho=0.6, budget=0.35, seed=11)
    in_b = [{k: v.to(dev) for k, v in si.make_layer(cfg_b, layer=0).items()}]
    stats_b = kvm.new_stats(dev)
    p_b = params(budget=cfg_b.budget)
    t_b = t_compress(p_b, inputs=in_b, stats_buf=stats_b)
    st_b = kvm.read_stats(stats_b)
    calls_b = min(reps, 50) + 3
    extras["budget_rule_case"] = {"rho": cfg_b.rho, "budget": cfg_b.budget, "compress_ms": t_b,
                                  "units_budget_rule_per_call": st_b.units_budget_rule / calls_b, "units": U,
                                  "mean_out_len": st_b.sum_out_len / (U * calls_b),
                                  "cap": int(math.floor(cfg_b.budget * cfg.seq))}
    del in_b
    # the whole path when the prefill attention already supplies the row log-sum-exp
    extras["compress_with_lse_ms"] = timed(
        lambda i: kvm.kvm_compress_with_lse(p, bufs[i % N_BUFFERS]["Q"], bufs[i % N_BUFFERS]["K"],
                                            bufs[i % N_BUFFERS]["V"], lses[i % N_BUFFERS], comp.K_out, comp.V_out,
                                            comp.out_len, comp.out_pos, None, None, ws, stream), min(reps, 50))
    # the prefill attention that hands over that log-sum-exp (Eq. 1 over the whole prompt), alone and followed
    # by the compression that uses its lse; and today's alternative, the same attention followed by kvm_compress
    o_att = torch.empty_like(b0["Q"])
    lse_att = torch.empty(cfg.batch, cfg.n_q_heads, cfg.seq, device=dev)
    def attend_then(i, with_lse):
        b = bufs[i % N_BUFFERS]
        kvm.kvm_prefill_attend(p, b["Q"], b["K"], b["V"], o_att, lse_att, None, stream)
        if with_lse is None:
            return
        kvm.kvm_compress_with_lse(p, b["Q"], b["K"], b["V"], lse_att if with_lse else None, comp.K_out, comp.V_out,
                                  comp.out_len, comp.out_pos, None, None, ws, stream)
    t_pre = timed(lambda i: attend_then(i, None), min(reps, 50))
    extras["prefill_attend_ms"] = t_pre
    extras["prefill_attend_tflops"] = 2 * work["flops_per_score_pass"] / (t_pre * 1e-3) / 1e12
    extras["prefill_attend_then_compress_with_lse_ms"] = timed(lambda i: attend_then(i, True), min(reps, 50))
    extras["prefill_attend_then_compress_ms"] = timed(lambda i: attend_then(i, False), min(reps, 50))
    ratio = torch.empty(U, device=dev)
    extras["layer_ratio_ms"] = timed(lambda i: kvm.kvm_layer_ratio(p, bufs[i % N_BUFFERS]["K"], ratio, None, ws,
                                                                   stream), min(reps, 50))
    extras["layer_ratio_mean"] = float(ratio.mean())
    qts = [b["Q"][:, :, -1].contiguous() for b in bufs]
    o_full = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, device=dev)
    o_comp = torch.empty_like(o_full)
    err = torch.empty(cfg.batch, cfg.n_q_heads, device=dev)
    ref = torch.empty_like(err)
    t_att = timed(lambda i: kvm.kvm_attend(p, qts[i % N_BUFFERS], bufs[i % N_BUFFERS]["K"], bufs[i % N_BUFFERS]["V"],
                                           cfg.seq, None, o_full, ws, stream), min(reps, 50))
    extras["attend_full_cache_ms"] = t_att
    extras["attend_full_cache_gbs"] = 2 * work["k_bytes"] / (t_att * 1e-3) / 1e9
    step(0)                                     # leave buffer 0's compressed cache in comp.*
    extras["output_perturbation_ms"] = timed(
        lambda i: kvm.kvm_output_perturbation(p, qts[0], b0["K"], b0["V"], comp.K_out, comp.V_out, comp.out_len,
                                              o_full, o_comp, err, ref, ws, stream), min(reps, 50))
    extras["output_perturbation_mean_rel"] = float((err / ref).mean())
    extras["l2_warm_ms_per_step"] = l2_warm

    # ---- end to end through the host-pointer entry point (pinned buffers, copies inside the timed region)
    pin = [{k: v.pin_memory() for k, v in h.items()} for h in host]
    dt = cfg.torch_dtype
    hK = torch.empty(cfg.batch, cfg.n_kv_heads, comp.cap, cfg.head_dim, dtype=dt).pin_memory()
    hV = torch.empty_like(hK).pin_memory()
    hlen = torch.empty(U, dtype=torch.int32).pin_memory()
    hpos = torch.empty(U * comp.cap, dtype=torch.int32).pin_memory()
    stage = torch.empty(kvm.kvm_host_staging_bytes(p), dtype=torch.uint8, device=dev)
    e2e_steps = max(3, min(args.steps, 50))

    def host_step(i):
        h = pin[i % N_BUFFERS]
        kvm.kvm_compress_host(p, h["Q"], h["K"], h["V"], hK, hV, hlen, hpos, stage, stream)

    for i in range(3):
        host_step(i)
    e2e_blocks = timed_blocks(host_step, e2e_steps, min_ms=min(300.0, args.min_ms), max_blocks=20)
    ms_e2e = sum(e2e_blocks) / len(e2e_blocks)
    assert int(hlen.sum()) > 0, "the host path returned no rows"
    esz = 2 if cfg.dtype == "bf16" else 4
    h2d = (cfg.batch * cfg.n_q_heads + 2 * U) * cfg.seq * cfg.head_dim * esz
    d2h = 2 * U * comp.cap * cfg.head_dim * esz + U * 4 + U * comp.cap * 4
    e2e = {"value": replicas.aggregate_throughput(world, e2e_steps, kv_tokens_per_step, ms_e2e), "unit": UNIT,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
           "ms_per_step": ms_e2e / e2e_steps, "blocks": len(e2e_blocks),
           "best_ms_per_step": min(e2e_blocks) / e2e_steps}
    del pin, stage, hK, hV

    # ---- the other workloads: a few layers each, generated layer by layer outside every timed region
    if pool is not None:
        from oracle import kvmo
        kvmo.lib()
        workloads = {}
        for name in OTHER_WORKLOADS:
            workloads[name] = bench_workload(kvm, kvmo, pool, name, dev, stream, peaks,
                                             with_cpu=not args.no_cpu_baseline)
        extras["workloads"] = workloads
        pool.close()
        pool.join()

    # ---- CPU baseline: the fp64 checker on this host's cores, rank 0, N = 1 only
    cpu = None
    if solo and not args.no_cpu_baseline:
        from oracle import kvmo
        kvmo.lib()                                   # load (and if need be compile) outside the timed region
        n_layers, t0 = 0, time.perf_counter()
        while n_layers < 3 or time.perf_counter() - t0 < 10.0:       # whole layers, about 10 s of CPU work
            h = host[n_layers % N_BUFFERS]
            kvmo.compress(h["Q"], h["K"], h["V"], float(np.float32(cfg.budget)), float(np.float32(0.17)),
                          float(np.float32(0.12)))
            n_layers += 1
        dtc = time.perf_counter() - t0
        cpu = {"value": n_layers * kv_tokens_per_step / dtc, "unit": UNIT, "cores": kvmo.num_threads(),
               "kind": "oracle", "sample": f"{n_layers} full {WORKLOAD} layers ({U} units each), {dtc:.2f} s"}

    if rank == 0:
        clocks = clk.summary()
        timing = {"blocks": len(block_ms), "steps_timed": len(block_ms) * args.steps,
                  "gpu_ms_timed": float(sum(block_ms)), "ms_per_step": per_step,
                  "ms_per_step_x_median_sm_mhz": (per_step["median"] * clocks["sm_mhz"]) if clocks["sm_mhz"] else None}
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "batch": cfg.batch, "heads": cfg.n_q_heads, "kv_heads": cfg.n_kv_heads,
                       "seq_len": cfg.seq, "head_dim": cfg.head_dim, "budget": cfg.budget, "layers_per_step": 1,
                       "l2": f"inputs larger than L2: {N_BUFFERS} rotating layer input sets of 100.7 MB",
                       "parallelism": f"replicas x{world} (independent layers per GPU, no collective)"},
            "clocks": clocks, "timing": timing, "e2e": e2e, "gpu_launches": 5 * len(block_ms) * args.steps,
            "roofline": roofline, "roofline_sfu": roofline_sfu, "kernels": kernels, "extras": extras,
            "path_roofline": {"roof_ms_per_step": t_roof_ms, "frac": e2e_frac,
                              "note": "slower of 2 score passes at bf16 peak and total bytes at HBM peak"},
            "cpu_baseline": cpu,
            "stats": {"mean_out_len": st.sum_out_len / max(1, U * n_calls),
                      "near_threshold_pairs_per_step": st.near_threshold / n_calls,
                      "units_budget_rule": st.units_budget_rule},
        }))
    if dist is not None:
        dist.destroy_process_group()


def bench_workload(kvm, kvmo, pool, name, dev, stream, peaks, with_cpu=True):
    """A few layers of one of the larger workloads: per-layer kvm_compress time (an event pair per layer), the
    all-layers throughput this implies, and the CPU checker on a sample of units with its all-units time
    extrapolated linearly (units are independent and of equal size)."""
    cfg = si.CONFIGS[name]
    layers = list(range(LAYERS_PER_WORKLOAD))
    host = generate_layers(pool, name, layers)
    bufs = [{k: v.to(dev) for k, v in h.items()} for h in host]
    p = kvm.make_params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq, cfg.head_dim, cfg.torch_dtype,
                        budget=cfg.budget)
    comp = kvm.Compressor(p, device=dev)
    stats = kvm.new_stats(dev)

    def call(b):
        kvm.kvm_compress(p, b["Q"], b["K"], b["V"], comp.K_out, comp.V_out, comp.out_len, comp.out_pos, None, stats,
                         comp.ws, stream)

    for b in bufs:
        call(b)
    torch.cuda.synchronize()
    times, total = [], 0.0
    while total < 200.0 and len(times) < 300:
        for b in bufs:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            call(b)
            e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
            total += times[-1]
    st = kvm.read_stats(stats)
    assert st.status == 0
    per_layer = stats_of(times)
    U = cfg.batch * cfg.n_kv_heads
    work = algorithmic_work(cfg)
    res = {
        "workload": cfg.name, "layers_timed": LAYERS_PER_WORKLOAD, "layers_in_model": cfg.layers,
        "inputs": "distinct layers in rotation (each larger than L2 together)", "ms_per_layer": per_layer,
        "kv_tokens_per_s_all_layers": U * cfg.seq / (per_layer["mean"] * 1e-3),
        "ms_all_layers": per_layer["mean"] * cfg.layers,
        "score_flops_over_call_time_tflops": 2 * work["flops_per_score_pass"] / (per_layer["mean"] * 1e-3) / 1e12,
        "path_roofline_frac": max(2 * work["flops_per_score_pass"] / (peaks["bf16_tflops"] * 1e12),
                                  (work["q_bytes"] + 2 * work["k_bytes"]) / (peaks["hbm_gbs"] * 1e9))
                              / (per_layer["mean"] * 1e-3),
        "mean_out_len": st.sum_out_len / (U * (len(times) + len(bufs))), "cap": comp.cap,
        "units_budget_rule_per_call": st.units_budget_rule / (len(times) + len(bufs)),
    }
    del bufs, comp
    torch.cuda.empty_cache()
    if with_cpu:
        # one whole query group for the GQA workload, eight units otherwise (first batch entry of layer 0)
        heads = [0] if cfg.group > 1 else list(range(8))
        d = si.make_layer(cfg, 0, batch_entries=[0], kv_heads=heads)
        recent, heavy = (0.17, 0.12) if cfg.budget >= 0.425 else (0.08, 0.02)
        t0 = time.perf_counter()
        kvmo.compress(d["Q"], d["K"], d["V"], float(np.float32(cfg.budget)), float(np.float32(recent)),
                      float(np.float32(heavy)))
        dtc = time.perf_counter() - t0
        res["cpu_checker"] = {
            "kind": "oracle", "cores": kvmo.num_threads(), "sample": f"{len(heads)} of {U} units of layer 0",
            "sample_seconds": dtc,
            "seconds_all_units_all_layers_extrapolated": dtc / len(heads) * U * cfg.layers,
            "kv_tokens_per_s_extrapolated": len(heads) * cfg.seq / dtc,
            "note": "extrapolated linearly from the sampled units",
        }
    return res


if __name__ == "__main__":
    main()
