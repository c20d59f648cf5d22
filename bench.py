#!/usr/bin/env python
"""Benchmark of the Swimba token-mixer forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config small_lm] [--impl ours|reference]

One "step" is one pass of the whole hot path (router, top-k, expert projection, mix, SSD) over one
batch of synthetic layer-shaped input.  Prints ONE JSON line on rank 0.  With N > 1 (torchrun)
every rank runs an independent replica on its own batch: the path has no exchange step, so there
is no collective on the data path (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2603_06938_b200 import replicas, synth

METRIC = "swimba_layer_fwd_tokens_per_s"
UNIT = "tokens/s"
NSETS = 4   # rotating input sets: together several times the 126 MB L2

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of each kernel from the ncu
# captures summarised under profiles/; None until a capture of that kernel exists.
NCU_TRAFFIC_BYTES = {
    # workload small_lm, one launch each (profiles/forward_small_lm_kernels.md); ncu flushes caches
    # before a launch and part of a kernel's writes can still sit in L2 when it ends
    # (the router launch includes the SSD step sizes; the projection reads the cleared rows it adds to;
    # the slot-mix and stand-alone step-size kernels do not run in this workload: no capture)
    "ssd_tiles": 82.547e6, "router_topk": 26.790e6, "expert_gemm": 36.986e6,
    # decode workload (profiles/decode_update_kernel.md)
    "decode_update": 479.8e6,
}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

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
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return dict(sm_mhz=statistics.median(sm) if sm else None,
                    sm_max_mhz=max(mx) if mx else None, reasons=sorted(reasons),
                    samples=len(sm))


def algorithmic_work(cfg: synth.LayerConfig, sm_count: int = 148):
    """Per-launch algorithmic work of each kernel for B x L tokens: bytes the method must move or
    flops it must execute, not what a particular kernel happens to do."""
    T, F, S, E, k = cfg.tokens, cfg.F, cfg.S, cfg.E, cfg.k
    H, P, N, G, Q = cfg.H, cfg.P, cfg.N, cfg.G, cfg.Q
    es = 2 if cfg.dtype == "bf16" else 4
    w = {}
    # below three 64-token tiles per SM the router launch also produces the SSD step sizes (dt in,
    # (Delta, log-decay) pairs out) of the bf16 tile path; above, they are a kernel of their own
    fused = E > 1 and cfg.dtype == "bf16" and F % 128 == 0 and -(-T // 64) < 3 * sm_count
    fused_scalars = T * H * 12 if fused else 0
    w["router_topk"] = dict(bound="hbm", work=T * F * es + E * F * es + T * k * 8 + fused_scalars)
    w["expert_gemm"] = dict(bound="tensor", work=2.0 * T * k * F * S)
    w["mix_slots"] = dict(bound="hbm", work=T * k * S * es + T * S * es)
    w["project_mix_simt"] = dict(bound="alu", work=2.0 * T * k * F * S)
    ssd_flops = float(T) * (Q * N * G + H * (Q * P + 4 * N * P))
    ssd_bytes = T * (2 * H * P * es + S * es + H * 4) + cfg.B * H * P * N * 4
    w["ssd_tiles"] = dict(bound="tensor", work=ssd_flops, bytes=ssd_bytes)
    w["ssd_sequential"] = dict(bound="alu", work=4.0 * T * H * P * N, bytes=ssd_bytes)
    w["segment_scan"] = dict(bound="hbm", work=0)
    w["ssd_scalars"] = dict(bound="hbm", work=T * H * 12)
    return w


def roofline_entry(name, avg_ms, work, pk):
    info = work.get(name)
    if info is None or avg_ms <= 0:
        return None
    if name == "ssd_tiles":
        # both roofs are close: report the one that binds (the larger ideal time), keep the other
        t_hbm = info["bytes"] / (pk["hbm_gbs"] * 1e9)
        t_tc = info["work"] / (pk["bf16_tflops"] * 1e12)
        ach_b = info["bytes"] / (avg_ms * 1e-3) / 1e9
        ach_f = info["work"] / (avg_ms * 1e-3) / 1e12
        ent = dict(kernel=name, traffic=NCU_TRAFFIC_BYTES.get(name), peak_source=pk["source"],
                   avg_ms=avg_ms, hbm_frac=ach_b / pk["hbm_gbs"], tensor_frac=ach_f / pk["bf16_tflops"])
        if t_hbm >= t_tc:
            ent.update(bound="hbm", achieved=ach_b, peak=pk["hbm_gbs"], unit="GB/s",
                       frac=ach_b / pk["hbm_gbs"])
        else:
            ent.update(bound="tensor", achieved=ach_f, peak=pk["bf16_tflops"], unit="TFLOP/s",
                       frac=ach_f / pk["bf16_tflops"])
        return ent
    if info["bound"] == "hbm":
        ach = info["work"] / (avg_ms * 1e-3) / 1e9
        peak, unit = pk["hbm_gbs"], "GB/s"
    elif info["bound"] == "tensor":
        ach = info["work"] / (avg_ms * 1e-3) / 1e12
        peak, unit = pk["bf16_tflops"], "TFLOP/s"
    else:
        # plain FP32 ALU work: 148 SMs x 128 FMA lanes x 2 flop x 1.965 GHz
        ach = info["work"] / (avg_ms * 1e-3) / 1e12
        peak, unit = 148 * 128 * 2 * 1.965e9 / 1e12, "TFLOP/s"
    return dict(kernel=name, bound=info["bound"], achieved=ach, peak=peak, unit=unit,
                frac=ach / peak, traffic=NCU_TRAFFIC_BYTES.get(name),
                peak_source=pk["source"], avg_ms=avg_ms)


def time_oracle_sample(cfg: synth.LayerConfig, n_seq: int, seed: int = 0):
    """The CPU oracle, as it stands, on n_seq whole sequences of the workload."""
    import dataclasses
    import oracle
    sub = dataclasses.replace(cfg, B=n_seq)
    inp = synth.make_inputs(sub, seed=seed)
    args = [synth.f64(inp[n]) for n in ("u", "x", "dt", "W_r", "W_e", "A", "dt_bias", "D")]
    t0 = time.perf_counter()
    oracle.swimba_forward(*args, k=cfg.k, G=cfg.G)
    dt = time.perf_counter() - t0
    return dict(value=sub.tokens / dt, unit=UNIT, cores=oracle.num_threads(), kind="oracle",
                sample=f"{n_seq} of {cfg.B} sequences x {cfg.L} tokens of {cfg.name}, fp64, "
                       f"{dt:.2f} s"), dt


def time_layer(sb, cfg, steps, warmup, n_sets=2, seed0=5000, repeat=1):
    """ms per forward of one layer configuration through swimba_forward (device-resident inputs)."""
    dcode = sb.DTYPE_FP32 if cfg.dtype == "fp32" else sb.DTYPE_BF16
    h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, dcode)
    sets = [synth.make_inputs(cfg, seed=seed0 + i) for i in range(n_sets)]
    wts = {n: sets[0][n].cuda() for n in ("W_r", "W_e", "A", "dt_bias", "D")}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    dev = [dict(u=s_["u"].cuda(), x=s_["x"].cuda(), dt=s_["dt"].cuda()) for s_ in sets]
    y = torch.empty_like(dev[0]["x"])
    hf = torch.empty(cfg.B, cfg.H, cfg.P, cfg.N, device="cuda")
    ws = torch.empty(sb.swimba_workspace_bytes(h, cfg.B, cfg.L), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        d = dev[i % n_sets]
        for _ in range(repeat):
            sb.swimba_forward(h, w, d["u"], d["x"], d["dt"], None, cfg.B, cfg.L, y, hf, None, None, ws)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    return e0.elapsed_time(e1) / steps


def bench_comparators(sb, cfg, steps, warmup, ms_swimba):
    """The same shape as (1) a dense Mamba-2 layer: the library with E = k = 1 (no router, one
    projection), and (2) E separated SSMs: every expert's streams projected for every token and E
    independent SSD evaluations with E states (the readout sum over the active experts is left
    out, so the figure is a lower bound of that design's cost)."""
    import dataclasses
    dense = dataclasses.replace(cfg, name=cfg.name + "_dense", E=1, k=1)
    ms_dense = time_layer(sb, dense, steps, warmup)
    ms_sep = time_layer(sb, dense, steps, warmup, repeat=cfg.E)
    return {
        "dense_mamba2": {"ms_per_step": ms_dense, "swimba_over_dense": ms_swimba / ms_dense,
                         "how": "same library, E = k = 1"},
        "separated_ssm_E_fold": {"ms_per_step": ms_sep, "swimba_over_separated": ms_swimba / ms_sep,
                                 "how": f"{cfg.E} dense-layer passes back to back (one projection "
                                        f"and one SSD evaluation per expert), readout sum not counted"},
    }


def run_reference(args, cfg, rank, world):
    if rank != 0:
        return
    n_seq = 1
    vals, times = [], []
    for i in range(args.warmup + args.steps):
        r, dt = time_oracle_sample(cfg, n_seq, seed=i)
        if i >= args.warmup:
            vals.append(r)
            times.append(dt)
    tok = n_seq * cfg.L
    ms = 1e3 * sum(times) / len(times)
    value = tok / (ms * 1e-3)
    cb = dict(vals[-1])
    cb["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, sample=f"{n_seq} sequence(s) per step"),
        "cpu_baseline": cb,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def config_dict(cfg, **extra):
    d = {"workload": f"{cfg.name}: B={cfg.B} L={cfg.L} d_model={cfg.F} H={cfg.H} P={cfg.P} "
                     f"N={cfg.N} G={cfg.G} E={cfg.E} top_k={cfg.k} chunk={cfg.Q} {cfg.dtype}",
         "tokens_per_step_per_gpu": cfg.tokens,
         "l2_policy": f"inputs rotate over {NSETS} distinct sets (> L2) between timed steps"}
    d.update(extra)
    return d


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", default="small_lm", choices=[c for c in synth.CONFIG_ORDER if c != "decode"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--decode-steps", type=int, default=512,
                    help="consecutive steps timed by the decode leg (the workload has 512)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-comparators", action="store_true")
    ap.add_argument("--no-e2e", action="store_true",
                    help="skip the host-buffer leg (for profiler launch lists of the device-resident steps)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = synth.CONFIGS[args.config]
    rank, world, local = replicas.rank_env()

    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return

    from paper_2603_06938_b200 import binding as sb
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    pk = peaks()
    dcode = sb.DTYPE_FP32 if cfg.dtype == "fp32" else sb.DTYPE_BF16
    h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, dcode)
    sets = [synth.make_inputs(cfg, seed=replicas.replica_seed(rank, i)) for i in range(NSETS)]
    wts = {n: sets[0][n].cuda() for n in ("W_r", "W_e", "A", "dt_bias", "D")}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    dev_sets = [dict(u=s["u"].cuda(), x=s["x"].cuda(), dt=s["dt"].cuda()) for s in sets]
    B, L = cfg.B, cfg.L
    y = torch.empty_like(dev_sets[0]["x"])
    hf = torch.empty(B, cfg.H, cfg.P, cfg.N, device="cuda")
    ws = torch.empty(sb.swimba_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        s = dev_sets[i % NSETS]
        sb.swimba_forward(h, w, s["u"], s["x"], s["dt"], None, B, L, y, hf, None, None, ws)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # the clock sampler is up before the warm-up, so that the warm-up steps run right in front of
    # the timed ones (no idle gap in which the GPU could leave its boost state)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    for i in range(args.warmup):
        step(i)
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    launches_per_step = sb.swimba_last_launch_count(h)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    ms_total = replicas.max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    ms_step = ms_total / args.steps
    value = replicas.whole_job_throughput(world, cfg.tokens, ms_step)

    # per-kernel durations, live, same launch configuration (CUDA events around every kernel)
    sb.swimba_profile(h, True)
    per = {}
    for i in range(args.steps):
        # two calls back to back, the second one is read: its first kernel then starts behind a
        # busy GPU, as in the timed loop, instead of absorbing the host's launch latency
        step(i)
        step(i + 1)
        for name, ms in sb.swimba_profile_read(h):
            per.setdefault(name, []).append(ms)
    sb.swimba_profile(h, False)
    clocks = sampler.stop() if rank == 0 else None

    work = algorithmic_work(cfg, torch.cuda.get_device_properties(local).multi_processor_count)
    tot = sum(sum(v) for v in per.values())
    kernels = []
    for name, v in per.items():
        n_per_step = len(v) / args.steps
        # a kernel launched several times per step (the two SSD passes of segmented sequences) is
        # rated on its time per step: the algorithmic work is per step
        ms_per_step_k = sum(v) / args.steps
        ent = roofline_entry(name, ms_per_step_k, work, pk) or dict(kernel=name, avg_ms=ms_per_step_k)
        ent["avg_ms"] = sum(v) / len(v)
        ent["ms_per_step"] = ms_per_step_k
        ent["share"] = sum(v) / tot if tot > 0 else 0.0
        ent["launches_per_step"] = n_per_step
        npos = int(round(n_per_step))
        if npos > 1 and len(v) % npos == 0:
            ent["per_launch_ms"] = [sum(v[i::npos]) / (len(v) // npos) for i in range(npos)]
        kernels.append(ent)
    kernels.sort(key=lambda e: -e["share"])
    dom = kernels[0] if kernels else None
    roofline = None
    if dom and "bound" in dom:
        roofline = {k_: dom[k_] for k_ in ("bound", "achieved", "peak", "unit", "frac", "traffic")}
        roofline["kernel"] = dom["kernel"]
        roofline["peak_source"] = "of " + pk["source"]

    e2e = None
    hws = None
    if not args.no_e2e:
        # end to end through the host-buffer entry point: pinned host inputs, H2D and D2H in the timed region
        hws = torch.empty(sb.swimba_host_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
        host_sets = [dict(u=s["u"].pin_memory(), x=s["x"].pin_memory(), dt=s["dt"].pin_memory())
                     for s in sets[:2]]
        y_host = torch.empty_like(sets[0]["x"]).pin_memory()
        for i in range(2):
            s = host_sets[i % 2]
            sb.swimba_forward_host(h, w, s["u"], s["x"], s["dt"], B, L, y_host, None, None, None, hws)
        barrier()
        e0.record(stream)
        for i in range(args.steps):
            s = host_sets[i % 2]
            sb.swimba_forward_host(h, w, s["u"], s["x"], s["dt"], B, L, y_host, None, None, None, hws)
        e1.record(stream)
        barrier()
        e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        es = 2 if cfg.dtype == "bf16" else 4
        h2d = cfg.tokens * (cfg.F * es + cfg.H * cfg.P * es + cfg.H * 4)
        d2h = cfg.tokens * cfg.H * cfg.P * es
        e2e = {"value": replicas.whole_job_throughput(world, cfg.tokens, e2e_ms / args.steps), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}
    sb.swimba_destroy(h)
    del dev_sets, hws, ws, y, hf

    decode = None
    if rank == 0 and world == 1 and not args.no_decode:
        decode = bench_decode(sb, pk, steps=args.decode_steps)

    comparators = None
    if rank == 0 and world == 1 and not args.no_comparators:
        comparators = bench_comparators(sb, cfg, args.steps, args.warmup, ms_step)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu, _ = time_oracle_sample(cfg, cfg.B)

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
            "data": "synthetic", "config": config_dict(cfg), "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "roofline": roofline,
            "kernels": kernels, "decode": decode, "comparators": comparators, "cpu_baseline": cpu,
        }
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def bench_decode(sb, pk, steps: int = 512, warmup: int = 8):
    """Decode configuration: us/step over `steps` consecutive steps, against the HBM bytes of the
    fp32 state read-modify-write."""
    cfg = synth.CONFIGS["decode"]
    h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, sb.DTYPE_BF16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(4)
    wt = synth.make_weights(cfg, gen)
    wts = {n: v.cuda() for n, v in wt.items()}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    state = (0.1 * torch.randn(cfg.B, cfg.H, cfg.P, cfg.N, generator=gen)).cuda()
    toks = [{n: v.cuda() for n, v in synth.make_decode_step_inputs(cfg, gen).items()} for _ in range(8)]
    y = torch.empty_like(toks[0]["x"])
    ws = torch.empty(sb.swimba_decode_workspace_bytes(h, cfg.B), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        t = toks[i % len(toks)]
        sb.swimba_decode_step(h, w, t["u"], t["x"], t["dt"], state, cfg.B, y, None, None, ws)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / steps
    launches = sb.swimba_last_launch_count(h)
    sb.swimba_profile(h, True)
    per = {}
    for i in range(32):
        step(i)
        step(i + 1)
        for name, ms in sb.swimba_profile_read(h):
            per.setdefault(name, []).append(ms)
    sb.swimba_profile(h, False)
    assert sb.swimba_status(h) == 0
    state_bytes = 2 * cfg.B * cfg.H * cfg.P * cfg.N * 4
    upd_us = 1e3 * sum(per.get("decode_update", [0])) / max(1, len(per.get("decode_update", [])))
    out = {
        "workload": f"decode: B={cfg.B} d_model={cfg.F} H={cfg.H} P={cfg.P} N={cfg.N} E={cfg.E} "
                    f"top_k={cfg.k}, fp32 state {state_bytes // 2 / 1e6:.0f} MB (> L2)",
        "us_per_step": us, "steps": steps, "launches_per_step": launches,
        "tokens_per_s": cfg.B / (us * 1e-6),
        "kernel_us": {n: 1e3 * sum(v) / len(v) for n, v in per.items()},
        "roofline": {"kernel": "decode_update", "bound": "hbm",
                     "achieved": state_bytes / (upd_us * 1e-6) / 1e9 if upd_us > 0 else None,
                     "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": state_bytes / (upd_us * 1e-6) / 1e9 / pk["hbm_gbs"] if upd_us > 0 else None,
                     "traffic": NCU_TRAFFIC_BYTES.get("decode_update"),
                     "whole_step_frac": state_bytes / (us * 1e-6) / 1e9 / pk["hbm_gbs"]},
    }
    sb.swimba_destroy(h)
    return out


if __name__ == "__main__":
    main()
