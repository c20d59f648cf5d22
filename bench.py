#!/usr/bin/env python
"""Benchmark of the Swimba token-mixer forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config mid] [--impl ours|reference]

One "step" is one pass of the whole hot path (router, top-k, expert projection, mix, SSD) over one
batch of synthetic layer-shaped input.  Prints ONE JSON line on rank 0.  The headline workload is
`mid` (the largest single-GPU forward shape that is run beside the dense and separated
comparators); `small_lm` and `long_seq` ride along as compact records under "workloads", the
decode workload under "decode".  With N > 1 (torchrun) every rank runs an independent replica on
its own batch: the path has no exchange step, so there is no collective on the data path (weak
scaling).

Timing.  The K-step timed region (barrier + synchronize on both sides, CUDA events on the launching
stream, max over ranks) is repeated back to back until about 1.5 s have passed, so that the clock
sampler sees the load; the reported step time is the median round's.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
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
L2_BYTES = 126e6
TIMED_SECONDS = 1.5   # the K-step timed region is repeated until it has covered about this long

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of each kernel from the ncu
# captures summarised under profiles/, per workload; a (workload, kernel) pair without a capture of
# the current kernel reports null.  ncu flushes caches before a launch, and part of a kernel's
# writes can still sit in L2 when it ends.
NCU_TRAFFIC_BYTES = {
    # profiles/forward_small_lm_kernels.md (the router launch includes the SSD step sizes)
    "small_lm": {"router_topk": 26.790e6, "expert_gemm": 36.989e6, "ssd_tiles": 82.690e6},
    # profiles/forward_mid_kernels.md
    "mid": {"ssd_scalars": 8.413e6, "router_topk": 147.230e6, "expert_gemm": 256.823e6, "ssd_tiles": 584.555e6},
    # profiles/ssd_segmented_long_seq.md (the state-only pass is a kernel of its own)
    "long_seq": {"ssd_state": 306.343e6, "ssd_tiles": 619.930e6, "segment_scan": 17.834e6},
    # profiles/decode_step_kernels.md
    "decode": {"router_topk": 0.593e6, "project_small": 9.070e6, "decode_update": 479.990e6},
}


def ncu_traffic(workload, kernel):
    return NCU_TRAFFIC_BYTES.get(workload, {}).get(kernel)


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
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def mark(self):
        return time.time()

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the two marks (all samples without marks)."""
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, r in self.rows:
            if t_begin is not None and not (t_begin <= ts <= t_end + 0.05):
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                pw.append(float(r[2]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return dict(sm_mhz=statistics.median(sm) if sm else None,
                    sm_max_mhz=max(mx) if mx else None, reasons=sorted(reasons),
                    samples=len(sm), power_w_max=max(pw) if pw else None,
                    window="samples taken during the timed rounds of the headline workload")


def algorithmic_work(cfg: synth.LayerConfig, nseg: int = 1, sm_count: int = 148):
    """Per-step algorithmic work of each kernel for B x L tokens: bytes the method must move or
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
    # the state-only pass of segmented sequences: x, Btilde and the step sizes in, segment states out
    # (every segment but a sequence's last one)
    part = (nseg - 1) / nseg if nseg > 1 else 0.0
    w["ssd_state"] = dict(bound="hbm", work=part * T * (H * P * es + G * N * es + H * 4)
                          + (nseg - 1) * cfg.B * H * P * N * 4)
    w["ssd_sequential"] = dict(bound="alu", work=4.0 * T * H * P * N, bytes=ssd_bytes)
    # the scan reads every segment's local end state and writes the state entering it
    w["segment_scan"] = dict(bound="hbm", work=(2 * nseg - 1) * cfg.B * H * P * N * 4)
    w["ssd_scalars"] = dict(bound="hbm", work=T * H * 12)
    return w


def roofline_entry(workload, name, avg_ms, work, pk):
    info = work.get(name)
    if info is None or avg_ms <= 0:
        return None
    if name == "ssd_tiles":
        # both roofs are close: report the one that binds (the larger ideal time), keep the other
        t_hbm = info["bytes"] / (pk["hbm_gbs"] * 1e9)
        t_tc = info["work"] / (pk["bf16_tflops"] * 1e12)
        ach_b = info["bytes"] / (avg_ms * 1e-3) / 1e9
        ach_f = info["work"] / (avg_ms * 1e-3) / 1e12
        ent = dict(kernel=name, traffic=ncu_traffic(workload, name), peak_source=pk["source"],
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
                frac=ach / peak, traffic=ncu_traffic(workload, name),
                peak_source=pk["source"], avg_ms=avg_ms)


def time_oracle_sample(cfg: synth.LayerConfig, n_seq: int, seed: int = 0):
    """The CPU oracle, as it stands, on n_seq whole sequences of the workload."""
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


def input_sets_needed(cfg: synth.LayerConfig) -> int:
    """Distinct input sets to rotate over so that together they are several times the L2."""
    es = 2 if cfg.dtype == "bf16" else 4
    per_set = cfg.tokens * (cfg.F * es + cfg.H * cfg.P * es + cfg.H * 4)
    return max(2, min(8, math.ceil(4 * L2_BYTES / per_set)))


class Layer:
    """One layer configuration resident on the device: handle, weights, rotating inputs, outputs."""

    def __init__(self, sb, cfg: synth.LayerConfig, rank: int = 0, seed0: int = 0, n_sets=None):
        self.sb, self.cfg = sb, cfg
        dcode = sb.DTYPE_FP32 if cfg.dtype == "fp32" else sb.DTYPE_BF16
        self.h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, dcode)
        self.n_sets = n_sets or input_sets_needed(cfg)
        self.host_sets = [synth.make_inputs(cfg, seed=seed0 + replicas.replica_seed(rank, i))
                          for i in range(self.n_sets)]
        s0 = self.host_sets[0]
        self.wts = {n: s0[n].cuda() for n in ("W_r", "W_e", "A", "dt_bias", "D")}
        self.w = sb.make_weights(*(self.wts[n] for n in ("W_r", "W_e", "A", "dt_bias", "D")))
        self.dev = [dict(u=s["u"].cuda(), x=s["x"].cuda(), dt=s["dt"].cuda()) for s in self.host_sets]
        self.y = torch.empty_like(self.dev[0]["x"])
        self.hf = torch.empty(cfg.B, cfg.H, cfg.P, cfg.N, device="cuda")
        self.ws = torch.empty(sb.swimba_workspace_bytes(self.h, cfg.B, cfg.L), dtype=torch.uint8,
                              device="cuda")

    def step(self, i):
        d = self.dev[i % self.n_sets]
        c = self.cfg
        self.sb.swimba_forward(self.h, self.w, d["u"], d["x"], d["dt"], None, c.B, c.L, self.y, self.hf,
                               None, None, self.ws)

    def check(self):
        assert self.sb.swimba_status(self.h) == 0, self.sb.swimba_last_error(self.h)

    def close(self):
        self.sb.swimba_destroy(self.h)
        self.dev = self.ws = self.y = self.hf = None


def time_rounds(layer: Layer, steps: int, warmup: int, dist, min_seconds: float, repeat: int = 1):
    """Warm-up, then rounds of exactly `steps` steps, each bracketed by a barrier and a device
    synchronisation on both sides and timed with CUDA events on the launching stream; every
    round's time is the maximum over ranks.  Returns (median ms per step, [ms per step of every
    round], launches per step)."""
    stream = torch.cuda.current_stream()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def run(n, base):
        for i in range(n):
            for _ in range(repeat):
                layer.step(base + i)

    run(warmup, 0)
    layer.check()
    launches = layer.sb.swimba_last_launch_count(layer.h)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    run(steps, 0)
    e1.record(stream)
    barrier()
    first = replicas.max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
    rounds = [first / steps]
    n_more = int(min(2000, max(0, math.ceil(min_seconds * 1e3 / max(first, 1e-3)) - 1)))
    for r in range(n_more):
        barrier()
        e0.record(stream)
        run(steps, (r + 1) * steps)
        e1.record(stream)
        barrier()
        rounds.append(e0.elapsed_time(e1) / steps)
    if dist is not None and len(rounds) > 1:
        t = torch.tensor(rounds, dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        rounds = [float(v) for v in t.tolist()]
    layer.check()
    return statistics.median(rounds), rounds, launches


def kernel_breakdown(layer: Layer, n: int, pk, sm_count: int):
    """Per-kernel durations, live, same launch configuration: CUDA events around every kernel
    (swimba_profile), read from the second of two back-to-back calls, so that the call's first
    kernel starts behind a busy GPU as in the timed loop."""
    sb, cfg = layer.sb, layer.cfg
    sb.swimba_profile(layer.h, True)
    per = {}
    for i in range(n):
        layer.step(i)
        layer.step(i + 1)
        for name, ms in sb.swimba_profile_read(layer.h):
            per.setdefault(name, []).append(ms)
    sb.swimba_profile(layer.h, False)
    nseg = sb.swimba_ssd_segments(layer.h, cfg.B, cfg.L)
    work = algorithmic_work(cfg, nseg, sm_count)
    tot = sum(sum(v) for v in per.values())
    kernels = []
    for name, v in per.items():
        n_per_step = len(v) / n
        # a kernel launched several times per step (the two SSD passes of segmented sequences) is
        # rated on its time per step: the algorithmic work is per step
        ms_per_step_k = sum(v) / n
        ent = roofline_entry(cfg.name, name, ms_per_step_k, work, pk) or dict(kernel=name, avg_ms=ms_per_step_k)
        ent["avg_ms"] = sum(v) / len(v)
        ent["ms_per_step"] = ms_per_step_k
        ent["share"] = sum(v) / tot if tot > 0 else 0.0
        ent["launches_per_step"] = n_per_step
        npos = int(round(n_per_step))
        if npos > 1 and len(v) % npos == 0:
            ent["per_launch_ms"] = [sum(v[i::npos]) / (len(v) // npos) for i in range(npos)]
        kernels.append(ent)
    kernels.sort(key=lambda e: -e["share"])
    return kernels, nseg


def dense_ratio(sb, cfg, steps, warmup, ms_swimba, with_separated: bool):
    """The same shape as (1) a dense Mamba-2 layer: the library with E = k = 1 (no router, one
    projection), and (2) E separated SSMs: every expert's streams projected for every token and E
    independent SSD evaluations with E states (the readout sum over the active experts is left
    out, so the figure is a lower bound of that design's cost)."""
    dense = dataclasses.replace(cfg, name=cfg.name + "_dense", E=1, k=1)
    lay = Layer(sb, dense, seed0=5000, n_sets=2)
    ms_dense, _, _ = time_rounds(lay, steps, warmup, None, 0.3)
    out = {"dense_mamba2": {"ms_per_step": ms_dense, "swimba_over_dense": ms_swimba / ms_dense,
                            "how": "same library, E = k = 1"}}
    if with_separated:
        ms_sep, _, _ = time_rounds(lay, steps, warmup, None, 0.0, repeat=cfg.E)
        out["separated_ssm_E_fold"] = {
            "ms_per_step": ms_sep, "swimba_over_separated": ms_swimba / ms_sep,
            "how": f"{cfg.E} dense-layer passes back to back (one projection and one SSD "
                   f"evaluation per expert), readout sum not counted"}
    lay.close()
    return out


def compact_kernels(kernels):
    keep = ("kernel", "bound", "frac", "hbm_frac", "tensor_frac", "ms_per_step", "share",
            "launches_per_step", "per_launch_ms", "traffic")
    return [{k_: e[k_] for k_ in keep if k_ in e} for e in kernels]


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
    cb["sample"] = f"every step: {n_seq} of {cfg.B} sequences x {cfg.L} tokens of {cfg.name}, fp64"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg),
        "cpu_baseline": cb,
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def config_dict(cfg):
    return {"workload": f"{cfg.name}: B={cfg.B} L={cfg.L} d_model={cfg.F} H={cfg.H} P={cfg.P} "
                        f"N={cfg.N} G={cfg.G} E={cfg.E} top_k={cfg.k} chunk={cfg.Q} {cfg.dtype}",
            "tokens_per_step_per_gpu": cfg.tokens,
            "l2_policy": f"inputs rotate over {input_sets_needed(cfg)} distinct sets (> L2) between timed steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="mid", choices=[c for c in synth.CONFIG_ORDER if c != "decode"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--seconds", type=float, default=TIMED_SECONDS,
                    help="the K-step timed region is repeated until about this long has been timed")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--decode-steps", type=int, default=512,
                    help="consecutive steps timed by the decode leg (the workload has 512)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-comparators", action="store_true")
    ap.add_argument("--no-workloads", action="store_true",
                    help="skip the compact records of the other forward workloads")
    ap.add_argument("--no-serving", action="store_true",
                    help="skip the batch x input-length sweep of packed prefill and decode")
    ap.add_argument("--no-e2e", action="store_true",
                    help="skip the host-buffer leg (for profiler launch lists of the device-resident steps)")
    ap.add_argument("--only", default=None,
                    choices=["backward", "general", "block", "serving", "sharded"],
                    help="run one of the side records alone on --config's workload and print it (the line is "
                         "not a bench line; for profiler captures of those kernels)")
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
    if args.only:
        side = {"backward": lambda: bench_backward(sb, cfg, steps=max(1, min(args.steps, 5)), warmup=2),
                "general": lambda: bench_general(sb, cfg, steps=max(1, min(args.steps, 10)), warmup=2),
                "block": lambda: bench_block(sb, cfg, steps=max(1, min(args.steps, 10)), warmup=2),
                "serving": lambda: bench_serving(sb, steps=max(1, min(args.steps, 10)), warmup=2),
                "sharded": lambda: bench_shard(sb, steps=max(1, min(args.steps, 10)), warmup=2)}
        print(json.dumps({"only": args.only, "record": side[args.only]()}))
        return
    pk = peaks()
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count
    stream = torch.cuda.current_stream()

    layer = Layer(sb, cfg, rank=rank)
    # the clock sampler is up before the warm-up, so that the warm-up steps run right in front of
    # the timed ones (no idle gap in which the GPU could leave its boost state)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    t_begin = sampler.mark()
    ms_step, rounds, launches_per_step = time_rounds(layer, args.steps, args.warmup, dist, args.seconds)
    t_end = sampler.mark()
    value = replicas.whole_job_throughput(world, cfg.tokens, ms_step)
    kernels, nseg = kernel_breakdown(layer, max(args.steps, 20), pk, sm_count)
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None

    dom = kernels[0] if kernels else None
    roofline = None
    if dom and "bound" in dom:
        roofline = {k_: dom[k_] for k_ in ("bound", "achieved", "peak", "unit", "frac", "traffic")}
        roofline["kernel"] = dom["kernel"]
        roofline["peak_source"] = "of " + pk["source"]
        for k_ in ("hbm_frac", "tensor_frac"):
            if k_ in dom:
                roofline[k_] = dom[k_]

    e2e = None
    if not args.no_e2e:
        # end to end through the host-buffer entry point: pinned host inputs, H2D and D2H in the timed region
        B, L = cfg.B, cfg.L
        hws = torch.empty(sb.swimba_host_workspace_bytes(layer.h, B, L), dtype=torch.uint8, device="cuda")
        host_sets = [dict(u=s["u"].pin_memory(), x=s["x"].pin_memory(), dt=s["dt"].pin_memory())
                     for s in layer.host_sets[:2]]
        y_host = torch.empty_like(layer.host_sets[0]["x"]).pin_memory()

        def host_step(i):
            s = host_sets[i % 2]
            sb.swimba_forward_host(layer.h, layer.w, s["u"], s["x"], s["dt"], B, L, y_host, None, None,
                                   None, hws)

        for i in range(3):
            host_step(i)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            host_step(i)
        e1.record(stream)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        layer.check()
        es = 2 if cfg.dtype == "bf16" else 4
        h2d = cfg.tokens * (cfg.F * es + cfg.H * cfg.P * es + cfg.H * 4)
        d2h = cfg.tokens * cfg.H * cfg.P * es
        e2e = {"value": replicas.whole_job_throughput(world, cfg.tokens, e2e_ms / args.steps), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "how": "swimba_forward_host: pinned host u, x, dt in, y out, every step"}
        del hws, host_sets, y_host
    layer.close()
    del layer
    torch.cuda.empty_cache()

    single = rank == 0 and world == 1
    comparators = None
    if single and not args.no_comparators:
        comparators = dense_ratio(sb, cfg, args.steps, args.warmup, ms_step, with_separated=True)

    workloads = None
    if single and not args.no_workloads:
        workloads = {}
        for name in ("small_lm", "long_seq", "mid"):
            if name == cfg.name:
                continue
            c2 = synth.CONFIGS[name]
            lay = Layer(sb, c2)
            ms2, r2, l2 = time_rounds(lay, args.steps, args.warmup, None, 0.5)
            k2, nseg2 = kernel_breakdown(lay, max(args.steps, 20), pk, sm_count)
            lay.close()
            del lay
            torch.cuda.empty_cache()
            rec = {"workload": config_dict(c2)["workload"], "ms_per_step": ms2,
                   "value": c2.tokens / (ms2 * 1e-3), "unit": UNIT, "rounds": len(r2),
                   "launches_per_step": l2, "ssd_segments": nseg2, "kernels": compact_kernels(k2)}
            if not args.no_comparators:
                rec["swimba_over_dense"] = dense_ratio(sb, c2, args.steps, args.warmup, ms2, False)[
                    "dense_mamba2"]["swimba_over_dense"]
            workloads[name] = rec

    decode = None
    if single and not args.no_decode:
        decode = bench_decode(sb, pk, steps=args.decode_steps)

    serving = None
    if single and not args.no_serving:
        serving = bench_serving(sb)

    shard = None
    if single and not args.no_serving:
        shard = bench_shard(sb)

    backward = None
    general = None
    block = None
    if single and not args.no_serving:
        backward = {name: bench_backward(sb, synth.CONFIGS[name]) for name in ("small_lm", "mid")}
        general = {name: bench_general(sb, synth.CONFIGS[name]) for name in ("small_lm", "mid")}
        block = {name: bench_block(sb, synth.CONFIGS[name]) for name in ("small_lm", "mid")}

    cpu = None
    if single and not args.no_cpu_baseline:
        cpu, _ = time_oracle_sample(cfg, cfg.B)

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
            "data": "synthetic", "config": config_dict(cfg), "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "roofline": roofline,
            "timing": {"rounds": len(rounds), "steps_per_round": args.steps,
                       "ms_per_step_median": ms_step, "ms_per_step_min": min(rounds),
                       "ms_per_step_max": max(rounds),
                       "how": "value is the median over rounds of exactly `steps` steps each"},
            "ssd_segments": nseg,
            "kernels": kernels, "comparators": comparators, "workloads": workloads,
            "decode": decode, "serving": serving, "sequence_sharded": shard, "backward_weights": backward,
            "general_form": general, "block_forward": block,
            "cpu_baseline": cpu,
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
                     "traffic": ncu_traffic("decode", "decode_update"),
                     "whole_step_frac": state_bytes / (us * 1e-6) / 1e9 / pk["hbm_gbs"]},
    }
    sb.swimba_destroy(h)
    return out


def _timed_calls(fn, steps, warmup):
    stream = torch.cuda.current_stream()
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        fn(i)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def _kernel_ms(sb, h, fns):
    """Per-kernel milliseconds of one pass through the given calls (event-bracketed)."""
    sb.swimba_profile(h, True)
    per = {}
    for fn in fns:
        fn(0)
        torch.cuda.synchronize()
        for name, t in sb.swimba_profile_read(h):
            per[name] = per.get(name, 0.0) + t
    sb.swimba_profile(h, False)
    return per


def bench_general(sb, cfg, steps: int = 10, warmup: int = 3):
    """The general form of the layer (expert-specific SSM inputs): swimba_route_project_slots, then
    swimba_ssd_slots on given per-slot inputs, for one batch of the workload.  Not tuned: the state
    equation is evaluated as k chunked recurrences."""
    h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, sb.DTYPE_BF16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(31)
    wts = {n: v.cuda() for n, v in synth.make_weights(cfg, gen).items()}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], None)
    dgen = torch.Generator(device="cuda")
    dgen.manual_seed(32)
    B, L, T = cfg.B, cfg.L, cfg.tokens
    u = torch.randn(B, L, cfg.F, generator=dgen, device="cuda").bfloat16()
    x_slots = torch.randn(cfg.k, B, L, cfg.H, cfg.P, generator=dgen, device="cuda").bfloat16()
    dt = 0.5 * torch.randn(B, L, cfg.H, generator=dgen, device="cuda")
    BCs = torch.empty(T, cfg.k, cfg.S, dtype=torch.bfloat16, device="cuda")
    y = torch.empty(B, L, cfg.H, cfg.P, dtype=torch.bfloat16, device="cuda")
    hf = torch.empty(B, cfg.H, cfg.P, cfg.N, device="cuda")
    ws = torch.empty(sb.swimba_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
    ws2 = torch.empty(sb.swimba_ssd_slots_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")

    def first(i):
        sb.swimba_route_project_slots(h, w, u, T, BCs, None, None, ws)

    def second(i):
        sb.swimba_ssd_slots(h, w, x_slots, BCs, dt, None, B, L, y, hf, ws2)

    def step(i):
        first(i)
        second(i)

    ms = _timed_calls(step, steps, warmup)
    per = _kernel_ms(sb, h, [first, second])
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    return {"workload": config_dict(cfg)["workload"], "ms": ms, "tokens_per_s": cfg.tokens / (ms * 1e-3),
            "kernel_ms": per}


def bench_block(sb, cfg, steps: int = 10, warmup: int = 3, d_conv: int = 4):
    """The whole block around the mixer (swimba_block_forward: in-projection, convolution + SiLU,
    routing and projection, the recurrence, gated norm, out-projection) for one batch of the
    workload.  Not tuned: the linear maps run through the grouped projection with one expert."""
    h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, sb.DTYPE_BF16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(41)
    wts = {n: v.cuda() for n, v in synth.make_weights(cfg, gen).items()}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    dgen = torch.Generator(device="cuda")
    dgen.manual_seed(42)
    B, L = cfg.B, cfg.L
    D = cfg.H * cfg.P
    W_in = (torch.randn(2 * D + cfg.H, cfg.F, generator=dgen, device="cuda") / cfg.F ** 0.5).bfloat16()
    conv_w = 0.5 * torch.randn(D + cfg.S, d_conv, generator=dgen, device="cuda")
    conv_b = 0.1 * torch.randn(D + cfg.S, generator=dgen, device="cuda")
    norm_w = 1.0 + 0.1 * torch.randn(D, generator=dgen, device="cuda")
    W_out = (torch.randn(cfg.F, D, generator=dgen, device="cuda") / D ** 0.5).bfloat16()
    bw = sb.make_block_weights(W_in, conv_w, conv_b, norm_w, W_out, d_conv)
    u = torch.randn(B, L, cfg.F, generator=dgen, device="cuda").bfloat16()
    out = torch.empty_like(u)
    cst = torch.empty(B, d_conv - 1, D + cfg.S, dtype=torch.bfloat16, device="cuda")
    hf = torch.empty(B, cfg.H, cfg.P, cfg.N, device="cuda")
    ws = torch.empty(sb.swimba_block_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")

    def step(i):
        sb.swimba_block_forward(h, w, bw, u, None, None, B, L, out, cst, hf, None, None, ws)

    ms = _timed_calls(step, steps, warmup)
    per = _kernel_ms(sb, h, [step])
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    flops = 2.0 * cfg.tokens * cfg.F * (2 * D + cfg.H) + 2.0 * cfg.tokens * D * cfg.F
    return {"workload": config_dict(cfg)["workload"], "ms": ms, "tokens_per_s": cfg.tokens / (ms * 1e-3),
            "kernel_ms": per, "linear_map_flops": flops}


def bench_backward(sb, cfg, steps: int = 5, warmup: int = 2):
    """The gradients of the router and expert matrices (swimba_backward_weights) for one batch of the
    workload: ms per call and per kernel.  These kernels run on the CUDA cores and are not tuned."""
    h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, sb.DTYPE_BF16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(21)
    wts = {n: v.cuda() for n, v in synth.make_weights(cfg, gen).items()}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    dgen = torch.Generator(device="cuda")
    dgen.manual_seed(22)
    B, L = cfg.B, cfg.L
    u = torch.randn(B, L, cfg.F, generator=dgen, device="cuda").bfloat16()
    x = torch.randn(B, L, cfg.H, cfg.P, generator=dgen, device="cuda").bfloat16()
    dy = torch.randn(B, L, cfg.H, cfg.P, generator=dgen, device="cuda").bfloat16()
    dt = 0.5 * torch.randn(B, L, cfg.H, generator=dgen, device="cuda")
    dWr = torch.empty(cfg.E, cfg.F, device="cuda")
    dWe = torch.empty(cfg.E, cfg.S, cfg.F, device="cuda")
    ws = torch.empty(sb.swimba_backward_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        sb.swimba_backward_weights(h, w, u, x, dt, None, dy, B, L, dWr, dWe, None, ws)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    sb.swimba_profile(h, True)
    step()
    torch.cuda.synchronize()
    per = {}
    for name, t in sb.swimba_profile_read(h):
        per[name] = per.get(name, 0.0) + t
    sb.swimba_profile(h, False)
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    return {"workload": config_dict(cfg)["workload"], "ms": ms, "tokens_per_s": cfg.tokens / (ms * 1e-3),
            "kernel_ms": per}


def bench_shard(sb, ranks: int = 8, steps: int = 10, warmup: int = 3):
    """One rank's compute of the sequence-sharded forward: the long_seq workload cut into `ranks` runs
    of tokens, the two halves (swimba_shard_summary, swimba_shard_finish) timed on this device for one
    shard, with the other ranks' summaries standing in as given arrays (the all-gather itself, about
    1 MB per rank, is not in the figure)."""
    cfg = synth.CONFIGS["long_seq"]
    L = cfg.L // ranks
    h = sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k, cfg.Q, sb.DTYPE_BF16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(12)
    wts = {n: v.cuda() for n, v in synth.make_weights(cfg, gen).items()}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    dgen = torch.Generator(device="cuda")
    dgen.manual_seed(13)
    nsets = 6                         # 6 x 30 MB of inputs + outputs: above L2 together
    sets = [dict(u=torch.randn(cfg.B, L, cfg.F, generator=dgen, device="cuda").bfloat16(),
                 x=torch.randn(cfg.B, L, cfg.H, cfg.P, generator=dgen, device="cuda").bfloat16(),
                 dt=0.5 * torch.randn(cfg.B, L, cfg.H, generator=dgen, device="cuda")) for _ in range(nsets)]
    ys = [torch.empty_like(s_["x"]) for s_ in sets]
    ws = torch.empty(sb.swimba_shard_workspace_bytes(h, cfg.B, L), dtype=torch.uint8, device="cuda")
    st = torch.empty(cfg.B, cfg.H, cfg.P, cfg.N, device="cuda")
    dc = torch.empty(cfg.B, cfg.H, device="cuda")
    all_state = 0.01 * torch.randn(ranks, cfg.B, cfg.H, cfg.P, cfg.N, device="cuda")
    all_decay = torch.rand(ranks, cfg.B, cfg.H, device="cuda")
    he = torch.empty(cfg.B, cfg.H, cfg.P, cfg.N, device="cuda")
    stream = torch.cuda.current_stream()

    def step(i):
        s_ = sets[i % nsets]
        sb.swimba_shard_summary(h, w, s_["u"], s_["x"], s_["dt"], cfg.B, L, st, dc, None, None, ws)
        sb.swimba_shard_finish(h, w, s_["x"], None, all_state, all_decay, ranks - 1, ranks, cfg.B, L,
                               ys[i % nsets], he, ws)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    return {"workload": f"long_seq cut into {ranks} shards of {L} tokens; the last rank's shard",
            "ms_per_shard": ms, "tokens_per_s_per_rank": cfg.B * L / (ms * 1e-3),
            "exchange_bytes_per_rank": cfg.B * cfg.H * (cfg.P * cfg.N + 1) * 4,
            "note": "compute of one rank (summary + finish); the all-gather between the halves is not timed"}


def bench_serving(sb, steps: int = 10, warmup: int = 3):
    """Serving-shaped batches on the `mid` layer shape: packed prefill (swimba_forward_packed) over a
    sweep of batch size x input length plus one batch of mixed lengths, and the decode step over a
    sweep of batch sizes.  Device-resident inputs, CUDA events on the launching stream."""
    base = synth.CONFIGS["mid"]
    h = sb.swimba_create(base.F, base.H, base.P, base.N, base.G, base.E, base.k, base.Q, sb.DTYPE_BF16)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(9)
    wts = {n: v.cuda() for n, v in synth.make_weights(base, gen).items()}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    stream = torch.cuda.current_stream()
    dgen = torch.Generator(device="cuda")
    dgen.manual_seed(10)
    Tmax = 32768
    # two input sets, together above L2
    sets = [dict(u=torch.randn(Tmax, base.F, generator=dgen, device="cuda").bfloat16(),
                 x=torch.randn(Tmax, base.H, base.P, generator=dgen, device="cuda").bfloat16(),
                 dt=0.5 * torch.randn(Tmax, base.H, generator=dgen, device="cuda")) for _ in range(2)]
    y = torch.empty_like(sets[0]["x"])

    def timed(fn):
        for i in range(warmup):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    prefill = []
    mixes = [("B=%d L=%d" % (b, l), [l] * b) for b in (1, 8, 64) for l in (128, 1024, 4096) if b * l <= Tmax]
    lg = torch.Generator().manual_seed(11)
    mixed = [int(v) for v in torch.exp(torch.rand(48, generator=lg) * (math.log(4096) - math.log(16)) + math.log(16))]
    while sum(mixed) > Tmax:
        mixed.pop()
    mixes.append(("%d sequences, lengths log-uniform in [16, 4096]" % len(mixed), mixed))
    mixes.append(("one 16384-token prompt", [16384]))
    mixes.append(("one 16384-token prompt among 64 single-token sequences", [16384] + [1] * 64))
    mixes.append(("64 single-token sequences", [1] * 64))
    for name, lens in mixes:
        cu = [0]
        for v in lens:
            cu.append(cu[-1] + v)
        T = cu[-1]
        assert T <= Tmax, "the batch does not fit the input arrays"
        hf = torch.empty(len(lens), base.H, base.P, base.N, device="cuda")
        ws = torch.empty(sb.swimba_packed_workspace_bytes(h, cu), dtype=torch.uint8, device="cuda")

        def step(i, cu=cu, hf=hf, ws=ws):
            s_ = sets[i % 2]
            sb.swimba_forward_packed(h, w, s_["u"], s_["x"], s_["dt"], None, cu, y, hf, None, None, ws)

        ms = timed(step)
        prefill.append({"batch": name, "tokens": T, "ms": ms, "tokens_per_s": T / (ms * 1e-3),
                        "segments": sb.swimba_packed_segments(h, cu)})
        del hf, ws
    decode = []
    for B in (1, 8, 32, 128):
        state = 0.1 * torch.randn(B, base.H, base.P, base.N, device="cuda")
        ws = torch.empty(sb.swimba_decode_workspace_bytes(h, B), dtype=torch.uint8, device="cuda")
        yd = torch.empty(B, base.H, base.P, dtype=torch.bfloat16, device="cuda")

        def dstep(i, B=B, state=state, ws=ws, yd=yd):
            s_ = sets[i % 2]
            sb.swimba_decode_step(h, w, s_["u"][:B], s_["x"][:B], s_["dt"][:B], state, B, yd, None, None, ws)

        ms = timed(dstep)
        decode.append({"batch": B, "us_per_step": ms * 1e3, "tokens_per_s": B / (ms * 1e-3)})
        del state, ws, yd
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    return {"layer": f"d_model={base.F} H={base.H} P={base.P} N={base.N} E={base.E} top_k={base.k} bf16",
            "steps": steps, "prefill_packed": prefill, "decode": decode}


if __name__ == "__main__":
    main()
