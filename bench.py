#!/usr/bin/env python3
"""Benchmark of the DSLA hot path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input: the chunkwise
prefill of the prompt(s) followed by one decode step on the states the prefill produced.  The
default workload is the Llama2-7B-shaped layer (B=1, H=32, d=128, T=4096, bf16, chunk 64).  A
second section times the batched-decode workload (B=128, H=32, d=128, 32 independent layers,
256 steps) because decode tokens/s is the other half of the metric.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg5] [--impl ours|reference]

With N > 1 (under torchrun) every rank runs the same per-GPU workload on its own GPU: sequences
and layers are independent, so there is no data-path collective (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_09316_b200 import inputs as gen  # noqa: E402

FLOP_PER_TOKEN_HEAD = lambda d, C: 2 * C * (d + d) + 8 * d * d          # QK^T, PV, 2x QS, 2x K^T V (full squares)
PREFILL_BYTES_PER_TOKEN_HEAD = lambda d, es: 4 * d * es + 8             # q, k, v, o + two fp32 gates
DECODE_BYTES_PER_ROW_HEAD = lambda d, es: 4 * d * d * 4 + 4 * d * es + 8  # 2 states read+write, q k v o, gates


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm_gbs=j["hbm_gbs"], bf16_tflops=j["bf16_tflops"],
                    bf16_tflops_sustained=j.get("bf16_tflops_sustained", j["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._t = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _once(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
            else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}
        for bit, name in names.items():
            if r & bit:
                self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                break
            time.sleep(0.002)

    def start(self):
        if self.nv:
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()

    def stop(self):
        if self._t:
            self._stop.set()
            self._t.join()
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def visible_nvml_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def dist_env():
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    return rank, world, local


def max_over_ranks(x, world, device):
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def workload_spec(name, dense=None):
    if dense:      # "B,H,T": a dense bf16 batch of the cfg2 head size, for shape sweeps (parity tests cover such shapes)
        B, H, T = (int(x) for x in dense.split(","))
        return dict(seed=1900, B=B, H=H, d=128, T=T, dtype="bf16", chunk=64, lens=[T] * B)
    c = dict(gen.CONFIGS[name])
    if name in ("cfg2", "cfg3"):
        c["lens"] = [c["T"]] * c["B"]
    elif name == "cfg5":
        c["lens"] = gen.ragged_lengths(c["seed"], c["N"], c["lo"], c["hi"])
    else:
        raise SystemExit(f"workload {name} is not a prefill workload (cfg4 is always reported under 'decode')")
    return c


# --------------------------------------------------------------------------------------------
KERNEL_SOURCES = {   # the files whose change makes a stored DRAM-traffic figure stale
    "tensor": ["dsla_prefill_tc.cu", "dsla_prefill_summary.cu", "dsla_prefill_tc.cuh", "tc_utils.cuh"],
    "pair": ["dsla_prefill_tc_pair.cu", "dsla_prefill_summary.cu", "dsla_prefill_tc.cuh", "tc_utils.cuh"],
    "decode": ["dsla_decode.cu"],
    "gate": ["dsla_gate_project.cu", "tc_utils.cuh"],
}


def source_digest(kind):
    import hashlib
    h = hashlib.sha1()
    for f in KERNEL_SOURCES[kind]:
        h.update(open(os.path.join(ROOT, "paper_2506_09316_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:12]


def stored_traffic(kernel, workload):
    """DRAM bytes per launch from the table of ncu captures kept with the profile summaries; None when there is no
    row for this kernel and workload or when the kernel's sources have changed since the capture."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    if not os.path.exists(path):
        return None
    for line in open(path):
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if len(cells) >= 4 and cells[0] == kernel and cells[1] == workload:
            try:
                return float(cells[2]) if cells[3] == source_digest(kernel) else None
            except ValueError:
                return None
    return None


def time_prefill(dsla, spec, kernel, steps, warmup, dev, rank, peaks, with_decode_leg=False, min_seconds=0.0):
    """Times `steps` prefills of one workload (CUDA events per step on the launching stream, rotating input sets larger
    than L2).  With min_seconds the timed region is repeated until it has lasted that long (sustained figure)."""
    H, d, lens = spec["H"], spec["d"], spec["lens"]
    N, T_total, max_len = len(lens), int(sum(lens)), int(max(lens))
    dense = len(set(lens)) == 1
    bytes_per_set = T_total * H * PREFILL_BYTES_PER_TOKEN_HEAD(d, 2)
    n_sets = 1 if bytes_per_set > 4 * 126e6 else max(2, int(np.ceil(4 * 126e6 / bytes_per_set)))
    sets = [gen.make_packed_device(spec["seed"] + 17 * i + 1000 * rank, lens, H, d, torch.bfloat16, device=dev)
            for i in range(n_sets)]
    outs = [torch.empty_like(s.v) for s in sets]
    st = dsla.dsla_state_alloc(N, H, d, d, device=dev)
    ws_bytes = dsla.binding.dsla_prefill_workspace_bytes(T_total, N, max_len, H, d, torch.bfloat16, 64, kernel,
                                                        dense_T=max_len if dense else None)
    ws = torch.empty(max(ws_bytes, 1), dtype=torch.uint8, device=dev) if ws_bytes else None
    dec = gen.make_packed_device(spec["seed"] + 5, [1] * N, H, d, torch.bfloat16, device=dev)
    dec_o = torch.empty_like(dec.v)
    stream = torch.cuda.current_stream()

    def step(i, ev=None):
        s = sets[i % n_sets]
        if ev:
            ev[0].record(stream)
        dsla.dsla_prefill(s.q, s.k, s.v, s.g_hist, s.g_rec, s.gamma, st, o=outs[i % n_sets],
                          cu_seqlens=None if dense else s.cu_seqlens, max_seqlen=max_len, chunk=64,
                          impl=kernel, workspace=ws)
        if ev:
            ev[1].record(stream)
        if with_decode_leg:
            dsla.dsla_decode_step(dec.q, dec.k, dec.v, dec.g_hist, dec.g_rec, s.gamma, st, o=dec_o)
        if ev:
            ev[2].record(stream)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    res = dict(sets=sets, dec=dec, st=st, ws=ws, lens=lens, dense=dense, max_len=max_len, n_sets=n_sets,
               bytes_per_set=bytes_per_set, T_total=T_total, N=N, step=step)
    if min_seconds > 0:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 0
        e0.record(stream)
        t_host = time.perf_counter()
        while True:
            for i in range(steps):
                step(n + i)
            n += steps
            if n % (8 * steps) == 0:
                stream.synchronize()          # bound the launch queue; the GPU stays busy between checks for < 1 %
            if time.perf_counter() - t_host >= min_seconds:
                break
        e1.record(stream)
        torch.cuda.synchronize()
        res.update(n=n, total_ms=e0.elapsed_time(e1))
        return res
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    res["evs"] = evs
    return res


def prefill_numbers(T_total, H, d, ms, peaks, world=1):
    flops = T_total * H * FLOP_PER_TOKEN_HEAD(d, 64)
    nbytes = T_total * H * PREFILL_BYTES_PER_TOKEN_HEAD(d, 2)
    tf = flops / (ms * 1e-3) / 1e12
    return {"ms": ms, "tokens_per_s": world * T_total / (ms * 1e-3), "tflops": tf, "frac": tf / peaks["bf16_tflops"],
            "hbm_gbs": nbytes / (ms * 1e-3) / 1e9, "hbm_frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}


def extra_prefill_section(dsla, name, kernel, steps, dev, rank, peaks, dense=None):
    """A further prefill workload reported beside the headline one: median and best of the per-step event times."""
    spec = workload_spec(name, dense)
    r = time_prefill(dsla, spec, kernel, steps, 3, dev, rank, peaks)
    time.sleep(0.2)          # let the power state of the section before settle; the clocks of this section are sampled below
    sampler = ClockSampler(visible_nvml_index(dev.index or 0))
    sampler.start()
    for i in range(steps):
        r["step"](i, r["evs"][i])
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = [e[0].elapsed_time(e[1]) for e in r["evs"]]
    out = {"workload": f"{dense or name}: N={r['N']} H={spec['H']} d={spec['d']} T_total={r['T_total']}", "kernel": kernel, "steps": steps,
           "clocks": clocks,
           "median": prefill_numbers(r["T_total"], spec["H"], spec["d"], float(np.median(ms)), peaks),
           "best": prefill_numbers(r["T_total"], spec["H"], spec["d"], float(np.min(ms)), peaks)}
    del r
    torch.cuda.empty_cache()
    return out


def bench_ours(args):
    import paper_2506_09316_b200 as dsla
    rank, world, local = dist_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    spec = workload_spec(args.workload, args.dense)
    H, d = spec["H"], spec["d"]
    r = time_prefill(dsla, spec, args.kernel, args.steps, args.warmup, dev, rank, peaks, with_decode_leg=True)
    sets, dec, st, ws, lens, dense, max_len = r["sets"], r["dec"], r["st"], r["ws"], r["lens"], r["dense"], r["max_len"]
    N, T_total, n_sets, bytes_per_set, evs, step = r["N"], r["T_total"], r["n_sets"], r["bytes_per_set"], r["evs"], r["step"]
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(visible_nvml_index(local))
    barrier(world)
    torch.cuda.synchronize()
    launches0 = dsla.dsla_launch_count()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True)
    t_stop = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        step(i, evs[i])
    t_stop.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    barrier(world)
    launches = dsla.dsla_launch_count() - launches0
    total_ms = max_over_ranks(t_start.elapsed_time(t_stop), world, dev)
    per_step = [e[0].elapsed_time(e[1]) for e in evs]
    prefill_ms = float(np.mean(per_step))
    decode_leg_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    ms_per_step = total_ms / args.steps
    tokens_per_step = T_total + N
    value = world * tokens_per_step / (ms_per_step * 1e-3)

    kernel_name = "pair" if args.kernel == "pair" else "tensor"
    pn = prefill_numbers(T_total, H, d, prefill_ms, peaks)
    traffic = stored_traffic(kernel_name, args.dense or args.workload) if args.kernel != "simt" else None
    roofline = {"kernel": f"prefill ({'summary + ' if N * H < 148 else ''}main launch, --kernel {args.kernel})", "bound": "tensor",
                "achieved": pn["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": pn["frac"], "traffic": traffic,
                "algorithmic_bytes": bytes_per_set, "algorithmic_flops": T_total * H * FLOP_PER_TOKEN_HEAD(d, 64),
                "peak_source": f"{peaks['source']} burst bf16 (kernel timed alone between events)",
                "hbm_gbs": pn["hbm_gbs"], "hbm_frac": pn["hbm_frac"],
                "median_ms": float(np.median(per_step)), "best_ms": float(np.min(per_step))}

    # ---- the same prefill repeated for at least half a second in one timed region (clocks and power settle)
    sustained = None
    if not args.no_sustained:
        sampler2 = ClockSampler(visible_nvml_index(local))
        sampler2.start()
        rs = time_prefill(dsla, spec, args.kernel, 16, 3, dev, rank, peaks, min_seconds=args.sustained_seconds)
        ck = sampler2.stop()
        ms = max_over_ranks(rs["total_ms"], world, dev) / rs["n"]
        pn2 = prefill_numbers(T_total, H, d, ms, peaks, world)
        sustained = {"seconds": rs["total_ms"] * 1e-3, "prefills": rs["n"], "ms": ms, "tokens_per_s": pn2["tokens_per_s"],
                     "tflops": pn2["tflops"], "peak": peaks["bf16_tflops_sustained"], "frac": pn2["tflops"] / peaks["bf16_tflops_sustained"],
                     "peak_source": f"{peaks['source']} sustained bf16", "clocks": ck}
        del rs

    # ---- end to end through the host-buffer entry points (pinned host memory)
    e2e = None
    if not args.no_e2e:
        e2e = bench_e2e(dsla, sets[0], dec, st, ws, lens, dense, max_len, args, world, dev)
    del r, sets, dec, st, ws, step, evs
    torch.cuda.empty_cache()

    # ---- the other prefill workloads and the other tensor-core variant (rank 0 reports; every rank runs them)
    more = None
    if not args.no_more:
        more = {}
        other = "pair" if args.kernel != "pair" else "tensor"
        if not args.dense:
            more[f"{args.workload}_{other}"] = extra_prefill_section(dsla, args.workload, other, 10, dev, rank, peaks)
        more["dense_4x37x16384"] = extra_prefill_section(dsla, "cfg2", args.kernel, 10, dev, rank, peaks, dense="4,37,16384")
        for name in ("cfg3", "cfg5"):      # the heaviest section last
            if name != args.workload or args.dense:
                more[name] = extra_prefill_section(dsla, name, args.kernel, 5, dev, rank, peaks)

    decode = None
    if not args.no_decode:
        decode = bench_decode(dsla, args, peaks, world, dev, rank)
        if not args.no_more:
            decode["n_states"] = bench_decode_nstate(dsla, peaks, dev, rank)

    extensions = None
    if not args.no_more and not args.no_decode:
        extensions = bench_extensions(dsla, peaks, dev, rank)

    gate_producer = None
    if not args.no_gate:
        gate_producer = bench_gate_project(dsla, peaks, dev, rank)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu_baseline = time_oracle_sample(spec, lens, budget_s=args.cpu_seconds)

    if rank == 0:
        line = {
            "metric": "dsla_prefill_plus_decode_tokens_per_s", "value": value, "unit": "tokens/s (one layer)",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{'dense ' + args.dense if args.dense else args.workload}: DSLA layer prefill B={N} H={H} d={d} T={lens[0] if dense else 'ragged'} "
                                   f"(T_total={T_total}) bf16 chunk=64 + 1 decode token per sequence",
                       "kernel": args.kernel, "l2": f"rotating {n_sets} input sets ({n_sets * bytes_per_set / 1e6:.0f} MB > 126 MB L2)",
                       "parallelism": f"replicated x{world} (independent sequences, no collective)"},
            "prefill_only": {"value": world * T_total / (prefill_ms * 1e-3), "unit": "tokens/s (one layer)", "ms": prefill_ms},
            "decode_leg_ms": decode_leg_ms,
            "roofline": roofline, "prefill_sustained": sustained, "prefill_more": more, "decode": decode,
            "gate_producer": gate_producer, "extensions": extensions, "cpu_baseline": cpu_baseline, "e2e": e2e,
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def bench_e2e(dsla, s, dec, st, ws, lens, dense, max_len, args, world, dev):
    H, d = s.H, s.d
    N, T_total = len(lens), int(sum(lens))
    pin = lambda t: t.cpu().pin_memory()
    hq, hk, hv, hg1, hg2 = pin(s.q), pin(s.k), pin(s.v), pin(s.g_hist), pin(s.g_rec)
    ho = torch.empty_like(hv).pin_memory()
    dq, dk, dv_, dg1, dg2 = pin(dec.q), pin(dec.k), pin(dec.v), pin(dec.g_hist), pin(dec.g_rec)
    do = torch.empty_like(dv_).pin_memory()
    stg = torch.empty(dsla.dsla_prefill_staging_bytes(T_total, N, max_len, H, d, torch.bfloat16,
                                                      dense_T=max_len if dense else None), dtype=torch.uint8, device=dev)
    stg2 = torch.empty(dsla.dsla_decode_staging_bytes(N, H, d, torch.bfloat16), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        dsla.dsla_prefill_host(hq, hk, hv, hg1, hg2, s.gamma, st, ho, stg, cu_seqlens=None if dense else s.cu_seqlens,
                               max_seqlen=max_len, chunk=64, impl=args.kernel, workspace=ws)
        dsla.dsla_decode_step_host(dq, dk, dv_, dg1, dg2, s.gamma, st, do, stg2)
        stream.synchronize()          # the caller reads o here

    n = max(3, min(args.steps, 10))
    for _ in range(2):
        step()
    barrier(world)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(n):
        step()
    torch.cuda.synchronize()
    dt = max_over_ranks(time.perf_counter() - t0, world, dev)
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hg1, hg2, dq, dk, dv_, dg1, dg2))
    d2h = sum(t.numel() * t.element_size() for t in (ho, do))
    return {"value": world * (T_total + N) * n / dt, "unit": "tokens/s (one layer)", "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "steps": n, "ms_per_step": dt / n * 1e3,
            "api": "dsla_prefill_host + dsla_decode_step_host, pinned host buffers, stream sync per step"}


def bench_decode(dsla, args, peaks, world, dev, rank):
    """Batched decode: B=128, H=32, d=128, 32 independent layers, fp32 dual states (17.2 GB)."""
    c = gen.CONFIGS["cfg4"]
    B, H, d, L, R = c["B"], c["H"], c["d"], args.decode_layers or c["layers"], c["ring"]
    steps, warm = args.decode_steps, 3
    states = [dsla.dsla_state_alloc(B, H, d, d, device=dev) for _ in range(L)]
    g = torch.Generator(device=dev)
    g.manual_seed(c["seed"] + rank)
    for s in states:
        s.tensor.normal_(0.0, c["state_std"], generator=g)
    ring = gen.make_packed_device(c["seed"] + 1 + rank, [1] * (L * R * B), H, d, torch.bfloat16, device=dev)
    view = lambda t: t.view(L, R, B, *t.shape[1:])
    q, k, v, g1, g2 = map(view, (ring.q, ring.k, ring.v, ring.g_hist, ring.g_rec))
    o = torch.empty_like(v)
    stream = torch.cuda.current_stream()

    def step(i):
        r = i % R
        for l in range(L):
            dsla.dsla_decode_step(q[l, r], k[l, r], v[l, r], g1[l, r], g2[l, r], ring.gamma, states[l], o=o[l, r])

    for i in range(warm):
        step(i)
    barrier(world)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    per_launch_s = ms * 1e-3 / (steps * L)
    bytes_launch = B * H * DECODE_BYTES_PER_ROW_HEAD(d, 2)
    gbs = bytes_launch / per_launch_s / 1e9
    return {"workload": f"cfg4: B={B} H={H} d={d} layers={L} steps={steps} bf16 tokens, fp32 states "
                        f"({L * B * 2 * H * d * d * 4 / 1e9:.1f} GB >> L2), input ring of {R} steps per layer",
            "value": world * B * steps / (ms * 1e-3), "unit": f"tokens/s ({L}-layer stack)",
            "layer_tokens_per_s": world * B * steps * L / (ms * 1e-3), "ms_per_step": ms / steps,
            "gpu_launches": steps * L,
            "roofline": {"kernel": "decode", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": stored_traffic("decode", "cfg4") if B == 128 else None,
                         "algorithmic_bytes": bytes_launch, "peak_source": f"{peaks['source']} copy bandwidth",
                         "us_per_launch": per_launch_s * 1e6}}


def bench_decode_nstate(dsla, peaks, dev, rank):
    """Decode step of the n-state form, n = 1, 2, 4, 8: B=128, H=32, d=128, a stack of layers whose states total
    about 4 GB (>> L2), 32 steps; bytes per launch = n d^2 8 + inputs, against the measured copy bandwidth."""
    c = gen.CONFIGS["cfg4"]
    B, H, d = c["B"], c["H"], c["d"]
    out = {}
    for n in (1, 2, 4, 8):
        per_layer = B * n * H * d * d * 4
        L = max(2, int(4e9 // per_layer))
        states = [dsla.dsla_state_alloc_n(B, n, H, d, d, device=dev) for _ in range(L)]
        g = torch.Generator(device=dev)
        g.manual_seed(c["seed"] + 31 * n + rank)
        for s in states:
            s.tensor.normal_(0.0, c["state_std"], generator=g)
        inp = gen.make_packed_device(c["seed"] + 7 * n + rank, [1] * (L * B), H, d, torch.bfloat16, device=dev)
        view = lambda t: t.view(L, B, *t.shape[1:])
        q, k, v = map(view, (inp.q, inp.k, inp.v))
        gates = torch.sigmoid(torch.randn((L, n, B, H), generator=g, device=dev) * 0.5 + 3.0)
        w = torch.rand((H, n), generator=g, device=dev)
        o = torch.empty_like(v)
        stream = torch.cuda.current_stream()
        steps = 32

        def step():
            for l in range(L):
                dsla.dsla_nstate_decode_step(q[l], k[l], v[l], gates[l], w, states[l], o=o[l])

        for _ in range(3):
            step()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        per_launch_s = e0.elapsed_time(e1) * 1e-3 / (steps * L)
        nbytes = B * H * (2 * n * d * d * 4 + 4 * d * 2 + 4 * n)
        gbs = nbytes / per_launch_s / 1e9
        out[str(n)] = {"layers": L, "us_per_launch": per_launch_s * 1e6, "algorithmic_bytes": nbytes, "achieved": gbs,
                       "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"]}
        del states, inp, q, k, v, gates, o
        torch.cuda.empty_cache()
    return out


# --------------------------------------------------------------------------------------------
def bench_extensions(dsla, peaks, dev, rank):
    """The wider forms of the layer: gates per key channel (decode and prefill), a decode batch in which half of the rows
    belong to another layer type (row mask), n-state prefill.  Decode sections: B=128, H=32, d=128, a stack of layers whose
    states total about 4 GB (>> L2); prefill sections: the cfg2 shape (one sequence of 4096 tokens, 32 heads)."""
    c = gen.CONFIGS["cfg4"]
    B, H, d = c["B"], c["H"], c["d"]
    out = {}
    L = 7
    g = torch.Generator(device=dev)
    g.manual_seed(c["seed"] + 900 + rank)
    states = [dsla.dsla_state_alloc(B, H, d, d, device=dev) for _ in range(L)]
    for s_ in states:
        s_.tensor.normal_(0.0, c["state_std"], generator=g)
    inp = gen.make_packed_device(c["seed"] + 901 + rank, [1] * (L * B), H, d, torch.bfloat16, device=dev)
    view = lambda t: t.view(L, B, *t.shape[1:])
    q, k, v, gs1, gs2 = map(view, (inp.q, inp.k, inp.v, inp.g_hist, inp.g_rec))
    gv1 = torch.sigmoid(torch.randn((L, B, H, d), generator=g, device=dev) * 0.5 + 6.0)
    gv2 = torch.sigmoid(torch.randn((L, B, H, d), generator=g, device=dev) * 0.5 + 1.0)
    mask = (torch.arange(B, device=dev) % 2 == 0).to(torch.uint8)
    o = torch.empty_like(v)
    stream = torch.cuda.current_stream()

    def timed(fn, steps=32):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e-3 / steps

    def per_channel():
        for l in range(L):
            dsla.dsla_decode_step(q[l], k[l], v[l], gv1[l], gv2[l], inp.gamma, states[l], o=o[l])

    def masked():
        for l in range(L):
            dsla.dsla_decode_step(q[l], k[l], v[l], gs1[l], gs2[l], inp.gamma, states[l], o=o[l], row_mask=mask)

    t = timed(per_channel) / L
    nbytes = B * H * (4 * d * d * 4 + 4 * d * 2 + 2 * d * 4)
    out["decode_per_key_channel_gates"] = {"layers": L, "us_per_launch": t * 1e6, "algorithmic_bytes": nbytes, "achieved": nbytes / t / 1e9,
                                           "unit": "GB/s", "frac": nbytes / t / 1e9 / peaks["hbm_gbs"]}
    t = timed(masked) / L
    nbytes = (B // 2) * H * DECODE_BYTES_PER_ROW_HEAD(d, 2)
    out["decode_row_mask_half"] = {"layers": L, "us_per_launch": t * 1e6, "algorithmic_bytes": nbytes, "achieved": nbytes / t / 1e9,
                                   "unit": "GB/s", "frac": nbytes / t / 1e9 / peaks["hbm_gbs"],
                                   "note": "every other row masked: only the live rows' states move"}
    del states, inp, q, k, v, gs1, gs2, gv1, gv2, o
    torch.cuda.empty_cache()

    T = 4096
    pin = gen.make_packed_device(c["seed"] + 902 + rank, [T], H, d, torch.bfloat16, device=dev)
    st = dsla.dsla_state_alloc(1, H, d, d, device=dev)
    gc1 = torch.sigmoid(torch.randn((T, H, d), generator=g, device=dev) * 0.5 + 6.0)
    gc2 = torch.sigmoid(torch.randn((T, H, d), generator=g, device=dev) * 0.5 + 1.0)
    oo = torch.empty_like(pin.v)
    t = timed(lambda: dsla.dsla_prefill(pin.q, pin.k, pin.v, gc1, gc2, pin.gamma, st, o=oo, max_seqlen=T), steps=5)
    out["prefill_per_key_channel_gates"] = {"workload": f"N=1 H={H} d={d} T={T} bf16", "ms": t * 1e3, "tokens_per_s": T / t,
                                            "kernel": "token-by-token CUDA-core recurrence"}
    for n in (1, 2, 4, 8):
        stn = dsla.dsla_state_alloc_n(1, n, H, d, d, device=dev)
        gates = torch.sigmoid(torch.randn((n, T, H), generator=g, device=dev) * 0.5 + 3.0)
        w = torch.rand((H, n), generator=g, device=dev)
        ws = torch.empty(max(1, dsla.dsla_nstate_prefill_workspace_bytes(pin.q, pin.k, pin.v, gates, w, max_seqlen=T)), dtype=torch.uint8, device=dev)
        t = timed(lambda: dsla.dsla_nstate_prefill(pin.q, pin.k, pin.v, gates, w, stn, o=oo, max_seqlen=T, workspace=ws), steps=10)
        t2 = timed(lambda: dsla.dsla_nstate_prefill(pin.q, pin.k, pin.v, gates, w, stn, o=oo, max_seqlen=T, impl="simt"), steps=3)
        passes = max(1, n // 2)
        flops = T * H * passes * FLOP_PER_TOKEN_HEAD(d, 64)      # what the kernel executes: every pass is a full dual-state pass
        out[f"prefill_{n}_states"] = {"workload": f"N=1 H={H} d={d} T={T} bf16, scalar gates", "ms": t * 1e3, "tokens_per_s": T / t,
                                      "kernel": f"chunkwise tensor-core kernel, {passes} pass(es) of two states",
                                      "executed_tflops": flops / t / 1e12, "token_by_token_kernel_ms": t2 * 1e3}
        del stn, ws
    return out


def bench_gate_project(dsla, peaks, dev, rank):
    """The gate producer (logistic(x W^T + b) on the tensor cores) for the tokens of one prefill: HBM-bound on reading x once.
    Input sets rotate so that x comes from DRAM (the sets together exceed L2)."""
    out = {}
    H, D_model = 32, 4096
    for name, T in (("T4096", 4096), ("T65536", 65536)):
        n_sets = max(2, int(np.ceil(160e6 / (T * D_model * 2))) + 1)
        g = torch.Generator(device=dev).manual_seed(4200 + rank)
        xs = [torch.randn((T, D_model), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16) for _ in range(n_sets)]
        w = (torch.randn((2 * H, D_model), generator=g, device=dev, dtype=torch.float32) / 64.0).to(torch.bfloat16)
        b = torch.zeros(2 * H, device=dev, dtype=torch.float32)
        gh = torch.empty((T, H), device=dev, dtype=torch.float32)
        gr = torch.empty((T, H), device=dev, dtype=torch.float32)
        for i in range(3):
            dsla.dsla_gate_project(xs[i % n_sets], w, b, g_hist=gh, g_rec=gr)
        torch.cuda.synchronize()
        steps, per = 10, 10      # ten calls per event pair: a call is shorter than the host needs to enqueue it alone
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(steps):
            evs[i][0].record()
            for j in range(per):
                dsla.dsla_gate_project(xs[(i * per + j) % n_sets], w, b, g_hist=gh, g_rec=gr)
            evs[i][1].record()
        torch.cuda.synchronize()
        ms = [e[0].elapsed_time(e[1]) / per for e in evs]
        nbytes = T * D_model * 2 + 2 * H * D_model * 2 + 2 * T * H * 4
        med = float(np.median(ms))
        out[name] = {"T": T, "H": H, "D_model": D_model, "ctas": (T + 127) // 128, "median_us": med * 1e3, "best_us": float(np.min(ms)) * 1e3,
                     "algorithmic_bytes": nbytes, "achieved_gbs": nbytes / (med * 1e-3) / 1e9,
                     "frac_of_hbm_peak": nbytes / (med * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": stored_traffic("gate", name),
                     "tflops": 2.0 * T * 2 * H * D_model / (med * 1e-3) / 1e12}
        del xs
        torch.cuda.empty_cache()
    return out


def time_oracle_sample(spec, lens, budget_s=15.0):
    """Times the CPU checker, as it stands, on a bounded sample of the same workload: the first
    `heads` heads of the first sequences, all their tokens (units are independent)."""
    from oracle import dsla_oracle as orc
    H, d = spec["H"], spec["d"]
    cores = orc.default_threads()
    rate_guess = 1.5e4 * cores * (128 * 128) / (d * d)       # (token, head) units per second, refined below
    order = np.argsort(lens)[::-1]
    seq = int(order[len(order) // 2]) if len(lens) > 1 else 0    # a median-length sequence
    L = int(lens[seq])
    heads = int(max(1, min(H, round(budget_s * rate_guess / L))))
    heads = max(heads, min(H, cores)) if L * min(H, cores) / rate_guess < 4 * budget_s else heads
    inp = gen.make_packed(spec["seed"], [L], heads, d, torch.bfloat16)
    f = inp.as_f64()
    t0 = time.perf_counter()
    orc.prefill(f["q"], f["k"], f["v"], f["g_hist"], f["g_rec"], f["gamma"], nthreads=cores)
    dt = time.perf_counter() - t0
    return {"value": L * heads / H / dt, "unit": "tokens/s (one layer)", "cores": int(min(cores, heads)), "kind": "oracle",
            "seconds": dt, "sample": f"{heads} of {H} heads x {L} tokens of one sequence (fp64, token by token); "
                                     f"layer tokens/s = tokens x heads/{H} / time"}


def bench_reference(args):
    """Reference arm: the fp64 CPU checker, as it stands, on this arm's workload and metric."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    spec = workload_spec(args.workload, getattr(args, "dense", None))
    lens = spec["lens"]
    per = max(1.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    res = None
    for _ in range(max(0, args.warmup)):
        time_oracle_sample(spec, lens, budget_s=per / 4)
    vals, secs = [], 0.0
    for _ in range(max(1, args.steps)):
        res = time_oracle_sample(spec, lens, budget_s=per)
        vals.append(res["value"])
        secs += res["seconds"]
    value = float(np.mean(vals))
    T_total = int(sum(lens))
    line = {"impl": "reference", "metric": "dsla_prefill_plus_decode_tokens_per_s", "value": value,
            "unit": "tokens/s (one layer)", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": (T_total + len(lens)) / value * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{args.workload}: same layer shape; each step is a bounded sample ({res['sample']})"},
            "cpu_baseline": {"value": value, "unit": "tokens/s (one layer)", "cores": res["cores"], "kind": "oracle",
                             "sample": res["sample"]},
            "e2e": {"value": value, "unit": "tokens/s (one layer)", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg3", "cfg5"])
    ap.add_argument("--dense", default=None, metavar="B,H,T", help="shape sweep: a dense bf16 d=128 batch instead of --workload")
    ap.add_argument("--kernel", default="auto", choices=["auto", "simt", "tensor", "pair"])
    ap.add_argument("--decode-steps", type=int, default=256)
    ap.add_argument("--decode-layers", type=int, default=0, help="layers in the decode section (0 = the workload's 32); "
                    "smaller stacks exist for profiler captures")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--sustained-seconds", type=float, default=0.6)
    ap.add_argument("--no-sustained", action="store_true")
    ap.add_argument("--no-more", action="store_true", help="skip the further prefill workloads and the n-state decode section")
    ap.add_argument("--no-gate", action="store_true", help="skip the gate-producer section")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        bench_reference(args)
    else:
        bench_ours(args)


if __name__ == "__main__":
    main()
