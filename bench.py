#!/usr/bin/env python
"""Benchmark of the CHELA hot path on B200: chunked causal linear attention forward.

One "step" = one chela_linattn_fwd call (through the C ABI) over the sequence-length-sweep workload at
L = 16384: B*L = 262144 tokens, H = 16, d_k = d_v = 64, chunk 64, bf16 inputs, fp32 accumulate and output.
Prints ONE JSON line (rank 0) with tokens/s, the roofline fraction of the dominant kernel against the
measured HBM peak, the end-to-end figure with host buffers, the clock record and the timed CPU oracle.
Extra keys: "sweep" (every L of the sweep, same launch configuration), "config2" and "mixer".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
    torchrun --nproc-per-node N bench.py --gpus N ...      (independent replicas, no collective on the path)
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

TOTAL_TOKENS = 262144
H, D, CHUNK = 16, 64, 64
L_MAIN = 16384
SWEEP_L = (1024, 2048, 4096, 8192, 16384, 32768, 65536)
# algorithmic bytes per token-head: read Q, K, V (bf16) once, write O (fp32) once
BYTES_PER_TOKEN_HEAD = 3 * D * 2 + D * 4
METRIC = "linattn_fwd_tokens_per_s"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu capture
# summarised in profiles/linattn_sm100_L2048_B16_ncu_full.md: 294.8 MB for 32768 tokens (B=16, L=2048, same
# grid), scaled by tokens to the timed workload (traffic is proportional to tokens: every tile is read once)
NCU_TRAFFIC_BYTES_PER_TOKEN = 293.9e6 / 32768
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML while the benchmark runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period, self.samples, self._stop_evt = index, period_s, [], threading.Event()
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        while not self._stop_evt.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                self.samples.append((time.perf_counter(), mhz, reasons))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()

    def summary(self, t0: float, t1: float):
        if self.nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml_unavailable"], "samples": 0}
        nv = self.nv
        window = [s for s in self.samples if t0 <= s[0] <= t1]
        names = {"sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
                 "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80)}
        seen = sorted({n for _, _, r in window for n, bit in names.items() if r & bit})
        return {"sm_mhz": statistics.median([m for _, m, _ in window]) if window else None,
                "sm_max_mhz": self.max_mhz, "reasons": seen, "samples": len(window)}


def oracle_inputs(n_batches: int, L: int, seed: int = 1234):
    import numpy as np
    from paper_2406_08128_b200 import inputs
    return tuple(a.astype(np.float64) for a in inputs.qkv(seed, n_batches, L, H, D, D, "bf16"))


def time_oracle_sample(qkv64, budget_s: float = 0.0):
    """Times the float64 oracle (recurrent form, as it stands) on the given inputs, repeating the pass until
    ``budget_s`` seconds of CPU work have been spent.  Returns (tokens/s, seconds, passes, threads)."""
    import oracle
    q, k, v = qkv64
    tokens = q.shape[0] * q.shape[1]
    passes, total = 0, 0.0
    while True:
        t0 = time.perf_counter()
        oracle.linattn_recurrent(q, k, v)
        total += time.perf_counter() - t0
        passes += 1
        if total >= budget_s or passes >= 200:
            break
    return passes * tokens / total, total, passes, oracle.num_threads()


def run_reference(args):
    """--impl reference: the CPU oracle, timed on the host cores, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    nb = max(1, min(4, TOTAL_TOKENS // L_MAIN))
    data = oracle_inputs(nb, L_MAIN)
    times = []
    for i in range(args.warmup + args.steps):
        tps, dt, _, cores = time_oracle_sample(data)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = nb * L_MAIN / (ms * 1e-3)
    sample = "recurrent-form float64 oracle on %d of the %d batch rows of the step (B=%d, L=%d, H=%d, d=%d) per step" % (
        nb, TOTAL_TOKENS // L_MAIN, nb, L_MAIN, H, D)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Elapsed time of the slowest rank (one MAX all-reduce of a scalar; the only collective of the job)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_s(ms_step: float, world: int, tokens_per_rank: int) -> float:
    """Whole-job throughput of `world` independent replicas that each process tokens_per_rank per step."""
    return world * tokens_per_rank / (ms_step * 1e-3)


def mixer_flops_per_token(D_model: int, n_heads: int, gated: bool = False) -> float:
    """Algorithmic tensor flops of the token mixer per token: three (five with the gates) D x D projections and the
    attention tiles.  The attention kernels walk 64-token tiles whatever `chunk` says (the result does not depend on
    it), so the tile term is 4*64*d + 4*d*d per token-head for chunk = 64 and chunk = 128 alike."""
    d_head = D_model // n_heads
    return (5 if gated else 3) * 2 * D_model * D_model + n_heads * (4 * 64 * d_head + 4 * d_head * d_head)


def sweep_linearity(sweep):
    """Time vs L at fixed B*L: spread of the times around their mean and the log-log slope of per-sequence time
    against L (a method that is linear in L has slope 1 and a flat time at fixed tokens)."""
    import math
    ms = [e["ms"] for e in sweep]
    mean = sum(ms) / len(ms)
    xs = [math.log(e["L"]) for e in sweep]
    ys = [math.log(e["ms"] / e["B"]) for e in sweep]   # per-sequence time
    n = len(xs)
    mx, my = sum(xs) / n, sum(ys) / n
    slope = sum((x - mx) * (y - my) for x, y in zip(xs, ys)) / sum((x - mx) ** 2 for x in xs)
    lo, hi = min(ms) / mean - 1.0, max(ms) / mean - 1.0
    return {"loglog_slope_time_per_sequence_vs_L": slope, "mean_ms": mean, "spread_vs_mean": [lo, hi],
            "max_over_min": max(ms) / min(ms), "within_pm10pct_of_mean": bool(lo >= -0.10 and hi <= 0.10),
            "slope_within_1_pm_0p05": bool(abs(slope - 1.0) <= 0.05), "min_hbm_frac": min(e["hbm_frac"] for e in sweep)}


def workload_config():
    return {"workload": "linattn_fwd sweep point L=%d: B=%d, H=16, d_k=d_v=64, chunk=64, bf16 in, fp32 out" % (
                L_MAIN, TOTAL_TOKENS // L_MAIN),
            "B": TOTAL_TOKENS // L_MAIN, "L": L_MAIN, "H": H, "d_k": D, "d_v": D, "chunk": CHUNK,
            "l2": "inputs+outputs %.2f GB per step, larger than L2: no flush needed" % (BYTES_PER_TOKEN_HEAD * TOTAL_TOKENS * H / 1e9)}


def run_mixer_mode(args):
    """--mixer: one step = one chela_mixer_fwd call; prints one JSON line (tokens/s, share of the bf16 tensor peak)."""
    import torch
    from paper_2406_08128_b200 import build as _build, chela
    _build.build()
    mb, ml, md, mh, mc = (int(x) for x in args.mixer.split(","))
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    gen = torch.Generator(device=dev).manual_seed(2)
    x = torch.randn(mb, ml, md, device=dev, generator=gen).to(torch.bfloat16)
    w_s = torch.randn(md, 3, device=dev, generator=gen) / 3 ** 0.5
    k_l = torch.randn(md, ml, device=dev, generator=gen) * torch.exp(-0.001 * torch.arange(ml, device=dev))[None, :]
    w_q, w_k, w_v = [(torch.randn(md, md, device=dev, generator=gen) / md ** 0.5).to(torch.bfloat16) for _ in range(3)]
    ws = torch.zeros(chela.mixer_workspace_bytes(mb, ml, md, mh, mc), dtype=torch.uint8, device=dev)
    out = torch.empty(mb, ml, md, device=dev)
    spec = chela.longconv_prepare(k_l)   # the long kernels' spectra: weights do not change between steps
    step = lambda: chela.mixer_prepared_fwd(x, w_s, spec, w_q, w_k, w_v, mh, chunk=mc, out=out, workspace=ws)
    if args.gated:   # Eqs. 8, 13, 14: two more projections, gates applied in the attention kernel's store
        w_a, w_o = [(torch.randn(md, md, device=dev, generator=gen) / md ** 0.5 / 12).to(torch.bfloat16) for _ in range(2)]
        ws = torch.zeros(chela.mixer_gated_workspace_bytes(mb, ml, md, mh, mc), dtype=torch.uint8, device=dev)
        step = lambda: chela.mixer_prepared_fwd(x, w_s, spec, w_q, w_k, w_v, mh, w_a=w_a, w_o=w_o, chunk=mc, out=out, workspace=ws)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    if chela.async_status(ws) != chela.OK:
        raise RuntimeError("device-side wait timed out")
    ms = e0.elapsed_time(e1) / args.steps
    peaks, peak_kind = measured_peaks()
    d_head = md // mh
    flops_tok = mixer_flops_per_token(md, mh, gated=args.gated)
    achieved = flops_tok * mb * ml / (ms * 1e-3) / 1e12
    print(json.dumps({"metric": "mixer_fwd_tokens_per_s", "value": mb * ml / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "token mixer forward B=%d L=%d D=%d H=%d chunk=%d, bf16 in, fp32 out" % (mb, ml, md, mh, mc)},
                      "roofline": {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                   "frac": achieved / peaks["bf16_tflops"], "traffic": None, "peak_source": peak_kind,
                                   "note": "algorithmic flops (3 dense projections + attention tiles) over the whole call; "
                                           "the long convolution (fp32 FFT on the plain ALUs) is inside the time"}}))


def run_probe_mode(args):
    """--probe NAME: a few calls of one small operation (the case the committed ncu summaries of that kernel were
    captured on); prints one JSON line with its time.  NAME: shortconv, linattn_d128, decode_step, mixer_gated."""
    import torch
    from paper_2406_08128_b200 import build as _build, chela
    _build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    gen = torch.Generator(device=dev).manual_seed(7)
    rnd = lambda *shape, s=1.0: (torch.randn(shape, device=dev, generator=gen) * s)
    name = args.probe
    if name == "shortconv":       # config 3's activations: 67 MB in, 67 MB out
        x, w = rnd(4, 16384, 512).to(torch.bfloat16), rnd(512, 3, s=3 ** -0.5)
        y = torch.empty_like(x)
        step, work = (lambda: chela.shortconv_fwd(x, w, out=y)), "shortconv B=4 L=16384 D=512 width 3, bf16"
    elif name == "linattn_d128":  # plain bf16, d = 128: 32768 tokens x 8 heads
        q, k, v = (rnd(2, 16384, 8, 128, s=0.125).to(torch.bfloat16) for _ in range(3))
        o = torch.empty(2, 16384, 8, 128, device=dev)
        ws = torch.zeros(chela.linattn_workspace_bytes(2, 8, 16384, 128, 128, 128), dtype=torch.uint8, device=dev)
        step, work = (lambda: chela.linattn_fwd(q, k, v, chunk=128, out=o, workspace=ws)), "linattn_fwd B=2 L=16384 H=8 d=128, bf16 in, fp32 out"
    elif name == "decode_step":   # one token per sequence against the carried state
        q, k, v = (rnd(256, 16, 64, s=0.125).to(torch.bfloat16) for _ in range(3))
        states = [torch.zeros(256, 16, 64, 64, device=dev) for _ in range(3)]
        o, it = torch.empty(256, 16, 64, device=dev), [0]

        def step():
            chela.linattn_step(q, k, v, states[it[0] % 3], out=o)
            it[0] += 1
        work = "linattn_step B=256 H=16 d=64, fp32 state"
    elif name == "mixer_gated":   # a quarter of config 3
        mb, ml, md, mh = 1, 16384, 512, 8
        x = rnd(mb, ml, md).to(torch.bfloat16)
        w_s = rnd(md, 3, s=3 ** -0.5)
        k_l = rnd(md, ml) * torch.exp(-0.001 * torch.arange(ml, device=dev))[None, :]
        w = [rnd(md, md, s=md ** -0.5).to(torch.bfloat16) for _ in range(5)]
        ws = torch.zeros(chela.mixer_gated_workspace_bytes(mb, ml, md, mh, 64), dtype=torch.uint8, device=dev)
        spec, o = chela.longconv_prepare(k_l), torch.empty(mb, ml, md, device=dev)
        step = lambda: chela.mixer_prepared_fwd(x, w_s, spec, w[0], w[1], w[2], mh, w_a=w[3], w_o=w[4], out=o, workspace=ws)
        work = "gated mixer B=1 L=16384 D=512 H=8, bf16 in, fp32 out, spectra prepared"
    else:
        raise SystemExit("unknown probe %r" % name)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    print(json.dumps({"probe": name, "workload": work, "steps": args.steps, "ms_per_step": e0.elapsed_time(e1) / args.steps}))


def run_backward_mode(args):
    """--backward: one step = one chela_linattn_bwd call at the timed workload (normaliser on); one JSON line."""
    import torch
    from paper_2406_08128_b200 import build as _build, chela
    _build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    gen = torch.Generator(device=dev).manual_seed(3)
    B, L = args.tokens // args.L, args.L
    q, k, v, d_o = ((torch.randn((B, L, H, D), device=dev, generator=gen) * s).to(torch.bfloat16) for s in (0.125, 0.125, 0.125, 1.0))
    ws = torch.zeros(int(chela.lib().chela_linattn_bwd_workspace_bytes(B, H, L, D, D)), dtype=torch.uint8, device=dev)
    step = lambda: chela.linattn_bwd(q, k, v, d_o, workspace=ws)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    if chela.async_status(ws) != chela.OK:
        raise RuntimeError("device-side wait timed out")
    ms = e0.elapsed_time(e1) / args.steps
    peaks, peak_kind = measured_peaks()
    # minimum traffic of a backward pass: read q, k, v, d_o (bf16), write dq, dk, dv (fp32)
    alg = B * L * H * D * (4 * 2 + 3 * 4)
    print(json.dumps({"metric": "linattn_bwd_tokens_per_s", "value": B * L / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
                      "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": "linattn backward B=%d L=%d H=%d d=%d, bf16 in, fp32 gradients, normaliser on" % (B, L, H, D)},
                      "roofline": {"bound": "hbm", "achieved": alg / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None, "peak_source": peak_kind,
                                   "note": "algorithmic bytes of a one-pass backward (20 B per element) over the time of the "
                                           "four-launch pass, which itself moves 2.4 times as much"}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="chela", choices=["chela", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the sweep / config-2 / mixer / CPU-oracle extras")
    ap.add_argument("--tokens", type=int, default=TOTAL_TOKENS, help="B*L of the timed step (profiling captures use a smaller case)")
    ap.add_argument("--L", type=int, default=L_MAIN, help="sequence length of the timed step")
    ap.add_argument("--backward", action="store_true", help="time chela_linattn_bwd at the timed workload instead")
    ap.add_argument("--mixer", default=None, metavar="B,L,D,H,chunk",
                    help="time the whole token mixer (short conv, long conv, Q/K/V, attention) on this shape instead, "
                         "e.g. 4,16384,512,8,64 (config 3) or 8,8192,1024,8,128 (config 4); single GPU")
    ap.add_argument("--gated", action="store_true", help="with --mixer: the gated call (two more projections, gates in the attention store)")
    ap.add_argument("--probe", default=None, metavar="NAME",
                    help="run a few calls of one small operation (shortconv, linattn_d128, decode_step, mixer_gated): the cases "
                         "the committed ncu summaries were captured on")
    args = ap.parse_args()
    if args.probe:
        return run_probe_mode(args)
    if args.backward:
        run_backward_mode(args)
        return
    if args.mixer:
        return run_mixer_mode(args)
    if (args.tokens, args.L) != (TOTAL_TOKENS, L_MAIN):
        globals().update(TOTAL_TOKENS=args.tokens, L_MAIN=args.L)
        args.no_extras = True
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2406_08128_b200 import build as _build, chela

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    chela.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    B = TOTAL_TOKENS // L_MAIN
    gen = torch.Generator(device=dev).manual_seed(100 + 14 + rank)
    flat = [(torch.randn(TOTAL_TOKENS * H * D, device=dev, generator=gen) * 0.125).to(torch.bfloat16) for _ in range(3)]
    out_flat = torch.empty(TOTAL_TOKENS * H * D, device=dev, dtype=torch.float32)
    ws_bytes = max([chela.linattn_workspace_bytes(max(TOTAL_TOKENS // L, 1), H, L, D, D, CHUNK) for L in SWEEP_L + (L_MAIN,)]
                   + [chela.linattn_workspace_bytes(8, 8, 4096, D, D, CHUNK)])
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)

    def views(L):
        b = TOTAL_TOKENS // L
        return [t.view(b, L, H, D) for t in flat], out_flat.view(b, L, H, D)

    def step(L):
        (q, k, v), o = views(L)
        chela.linattn_fwd(q, k, v, chunk=CHUNK, out_dtype=chela.F32, out=o, workspace=ws)

    kind = chela.linattn_kernel_kind(B, H, L_MAIN, D, D, CHUNK)
    sampler = ClockSampler(local)
    sampler.start()

    # ---- timed region: exactly K steps, CUDA events on the launching stream ---------------------------
    for _ in range(args.warmup):
        step(L_MAIN)
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.perf_counter()
    ev0.record()
    for _ in range(args.steps):
        step(L_MAIN)
    ev1.record()
    barrier()
    t_wall1 = time.perf_counter()
    ms_total = ev0.elapsed_time(ev1)
    if chela.async_status(ws) != chela.OK:
        raise RuntimeError("device-side wait timed out during the timed region")
    # the clock the hardware counts (SM cycles over global-timer nanoseconds), right after the timed region
    sm_mhz_counted = chela.debug_sm_clock_mhz()
    # keep the GPU under the same load a little longer if the timed region was too short to sample clocks
    clocks = sampler.summary(t_wall0, t_wall1)
    if clocks["samples"] < 5:
        t_b0 = time.perf_counter()
        while time.perf_counter() - t_b0 < 0.5:
            for _ in range(20):
                step(L_MAIN)
            torch.cuda.synchronize()
        clocks = sampler.summary(t_wall0, time.perf_counter())
        clocks["note"] = "timed region too short for NVML polling: window extended over an identical untimed burst"
    clocks["sm_mhz_counted"] = sm_mhz_counted
    ms_step = max_over_ranks(ms_total, world, dev) / args.steps
    value = job_tokens_per_s(ms_step, world, TOTAL_TOKENS)

    # ---- end to end: host buffers in, host buffer out, through the same C-ABI call ---------------------
    host_in = [torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for x in flat]
    host_out = torch.empty(out_flat.shape, dtype=out_flat.dtype, pin_memory=True)
    e2e_steps = max(2, min(args.steps, 5))

    # Every step copies all of its inputs host -> device and all of its output device -> host.  The batch is
    # cut into slices of batch rows (independent problems); a copy-in stream, the compute stream and a
    # copy-out stream run one slice apart, so the step costs about the slowest of the three legs (PCIe).
    B_full = TOTAL_TOKENS // L_MAIN
    n_slices = 4 if B_full % 4 == 0 else 1
    rows = B_full // n_slices
    per = rows * L_MAIN * H * D
    s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    ws_slices = [torch.zeros(max(chela.linattn_workspace_bytes(rows, H, L_MAIN, D, D, CHUNK), 16), dtype=torch.uint8, device=dev)
                 for _ in range(n_slices)]

    # Dependencies are tracked per slice and carried from step to step, so the copy engines never drain between
    # steps: a slice's inputs are overwritten once the previous step's kernel on that slice has finished, its
    # output slice once the previous step's copy-out of it has finished.
    carried = {"cmp": [None] * n_slices, "out": [None] * n_slices}

    def e2e_step():
        for i in range(n_slices):
            sl = slice(i * per, (i + 1) * per)
            ev_in, ev_cmp, ev_out = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
            with torch.cuda.stream(s_in):
                if carried["cmp"][i] is not None:
                    s_in.wait_event(carried["cmp"][i])
                for d_, h_ in zip(flat, host_in):
                    d_[sl].copy_(h_[sl], non_blocking=True)
                ev_in.record(s_in)
            s_cmp.wait_event(ev_in)
            if carried["out"][i] is not None:
                s_cmp.wait_event(carried["out"][i])
            q, k, v = (t[sl].view(rows, L_MAIN, H, D) for t in flat)
            chela.linattn_fwd(q, k, v, chunk=CHUNK, out_dtype=chela.F32, out=out_flat[sl].view(rows, L_MAIN, H, D),
                              workspace=ws_slices[i])
            ev_cmp.record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp)
                host_out[sl].copy_(out_flat[sl], non_blocking=True)
                ev_out.record(s_out)
            carried["cmp"][i], carried["out"][i] = ev_cmp, ev_out

    def e2e_drain():   # the last step is over when its last output slice is on the host
        s_cmp.wait_stream(s_in)
        s_cmp.wait_stream(s_out)

    s_in.wait_stream(s_cmp)
    e2e_step()
    e2e_drain()
    barrier()
    ev0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e2e_drain()
    ev1.record()
    barrier()
    e2e_ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev) / e2e_steps
    e2e = {"value": job_tokens_per_s(e2e_ms, world, TOTAL_TOKENS), "unit": "tokens/s", "ms_per_step": e2e_ms,
           "steps": e2e_steps, "h2d_bytes_per_step": int(sum(x.numel() * x.element_size() for x in flat)),
           "d2h_bytes_per_step": int(out_flat.numel() * out_flat.element_size()),
           "pipelining": "%d batch slices per step; copy-in, compute and copy-out streams, dependencies per slice and carried "
                         "across steps (every step copies all its inputs in and all its output out)" % n_slices}
    for w_ in ws_slices:
        if chela.async_status(w_) != chela.OK:
            raise RuntimeError("device-side wait timed out in the end-to-end leg")
    del host_in, host_out, ws_slices

    peaks, peak_kind = measured_peaks()
    alg_bytes = BYTES_PER_TOKEN_HEAD * TOTAL_TOKENS * H
    achieved = alg_bytes / (ms_step * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES_PER_TOKEN * TOTAL_TOKENS,
                "traffic_source": "ncu capture of a 32768-token case scaled by tokens; a lower bound (the tail of the output is still "
                                  "in L2 when that small kernel ends), reads equal the algorithmic reads", "peak_source": peak_kind,
                "kernel": "linattn_sm100_kernel<64,float>" if kind == 2 else "linattn_simt_kernel",
                "algorithmic_bytes_per_launch": alg_bytes, "launch_ms": ms_step}

    line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(),
            "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps, "kernel_kind": kind, "roofline": roofline}

    def timed(fn, iters, warm=3):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(iters):
            fn()
        b_.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b_) / iters

    if rank == 0 and not args.no_extras:
        # ---- every L of the sweep, same kernel and launch path ---------------------------------------
        sweep = []
        for L in SWEEP_L:
            tw0 = time.perf_counter()
            ms = timed(lambda: step(L), 30, warm=5)
            ck = sampler.summary(tw0, time.perf_counter())   # the SM clock NVML reports for this point (warm-up included)
            # and the clock the hardware counts right after it: SM cycles over global-timer nanoseconds.  The two differ:
            # NVML was seen to report the maximum clock with no throttle reason while the counted clock had dropped to
            # 1400 MHz after a few hundred milliseconds of load, and the shapes with fewer sequences than SMs follow it.
            sweep.append({"L": L, "B": TOTAL_TOKENS // L, "ms": ms, "tokens_per_s": TOTAL_TOKENS / (ms * 1e-3),
                          "hbm_frac": alg_bytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "sm_mhz_nvml": ck["sm_mhz"],
                          "sm_mhz_counted": chela.debug_sm_clock_mhz(), "clock_reasons": ck["reasons"]})
        line["sweep"] = sweep
        line["sweep_linearity"] = sweep_linearity(sweep)
        # The same points again, each after a one-second pause: back to back, the counted SM clock falls from point to
        # point (1965 -> 1680 -> 1400-1580 MHz while NVML reports 1965), and the shapes with fewer sequences than SMs
        # follow it; rested, every point starts from the same clock state.  Both sets are printed; neither is the headline.
        rested = []
        for L in SWEEP_L:
            time.sleep(1.0)
            ms = timed(lambda: step(L), 30, warm=5)
            rested.append({"L": L, "B": TOTAL_TOKENS // L, "ms": ms, "tokens_per_s": TOTAL_TOKENS / (ms * 1e-3),
                           "hbm_frac": alg_bytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                           "sm_mhz_counted": chela.debug_sm_clock_mhz()})
        line["sweep_rested"] = rested
        line["sweep_rested_linearity"] = sweep_linearity(rested)
        # ---- d = 128 (config 4's head size) plain bf16 linear attention at the same token count: H = 8 ----------
        n128 = TOTAL_TOKENS * 8 * 128
        q8, k8, v8 = (flat[j][:n128].view(16, TOTAL_TOKENS // 16, 8, 128) for j in range(3))
        o8 = out_flat[:n128].view(16, TOTAL_TOKENS // 16, 8, 128)
        ws8 = torch.zeros(chela.linattn_workspace_bytes(16, 8, TOTAL_TOKENS // 16, 128, 128, 128), dtype=torch.uint8, device=dev)
        time.sleep(1.0)   # like the rested sweep: from the clock state of an idle GPU; the counted clock is printed
        ms = timed(lambda: chela.linattn_fwd(q8, k8, v8, chunk=128, out_dtype=chela.F32, out=o8, workspace=ws8), 20, warm=5)
        mhz128 = chela.debug_sm_clock_mhz()
        if chela.async_status(ws8) != chela.OK:
            raise RuntimeError("device-side wait timed out in the d = 128 extra")
        b128 = TOTAL_TOKENS * 8 * (3 * 128 * 2 + 128 * 4)
        line["linattn_d128"] = {"B": 16, "L": TOTAL_TOKENS // 16, "H": 8, "d": 128, "ms": ms, "tokens_per_s": TOTAL_TOKENS / (ms * 1e-3),
                                "hbm_frac": b128 / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "sm_mhz_counted": mhz128,
                                "note": "plain bf16 in, fp32 out, d_k = d_v = 128; algorithmic bytes 1280 per token-head; "
                                        "measured after a one-second pause"}
        del ws8
        # ---- config 2: B=8, H=8, L=4096 (134 MB in + 67 MB out; four rotating buffer sets exceed L2) ----
        sets = []
        for s in range(4):
            n = 8 * 4096 * 8 * 64
            sets.append(([flat[j][s * n:(s + 1) * n].view(8, 4096, 8, 64) for j in range(3)],
                         out_flat[s * n:(s + 1) * n].view(8, 4096, 8, 64)))
        state = {"i": 0}

        def c2():
            (q, k, v), o = sets[state["i"] % 4]
            state["i"] += 1
            chela.linattn_fwd(q, k, v, chunk=64, out_dtype=chela.F32, out=o, workspace=ws)

        ms = timed(c2, 40)
        mhz_c2 = chela.debug_sm_clock_mhz()
        time.sleep(1.0)
        ms_rested = timed(c2, 40)
        c2_bytes = BYTES_PER_TOKEN_HEAD * 8 * 4096 * 8
        line["config2"] = {"ms": ms, "tokens_per_s": 8 * 4096 / (ms * 1e-3),
                           "hbm_frac": c2_bytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "sm_mhz_counted": mhz_c2,
                           "ms_rested": ms_rested, "hbm_frac_rested": c2_bytes / (ms_rested * 1e-3) / 1e9 / peaks["hbm_gbs"],
                           "sm_mhz_counted_rested": chela.debug_sm_clock_mhz(),
                           "note": "ms: right after the other extras; ms_rested: after a one-second pause"}
        if chela.async_status(ws) != chela.OK:
            raise RuntimeError("device-side wait timed out in the extras")
        del sets
        # ---- token mixer forward (configs 3 and 4): short conv + SiLU, long conv, Q/K/V, attention --------
        # roofline: bf16 tensor peak over the algorithmic flops (3 dense projections + the attention tiles)
        # fp32 FMA rate of this GPU, measured now: a cuBLAS fp32 GEMM with TF32 off runs on the plain FMA pipes
        # (library kernel, used only as the denominator of the long convolution's ALU fraction)
        tf32_was = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = False
        ga, gb = torch.randn(8192, 8192, device=dev), torch.randn(8192, 8192, device=dev)
        ms_g = timed(lambda: torch.matmul(ga, gb), 5, warm=2)
        torch.backends.cuda.matmul.allow_tf32 = tf32_was
        fp32_peak = 2 * 8192.0 ** 3 / (ms_g * 1e-3) / 1e12
        del ga, gb
        mixers = []
        for (mb, ml, md, mh, mc) in ((4, 16384, 512, 8, 64), (8, 8192, 1024, 8, 128)):
            x = torch.randn(mb, ml, md, device=dev, generator=gen).to(torch.bfloat16)
            w_s = torch.randn(md, 3, device=dev, generator=gen) / 3 ** 0.5
            k_l = torch.randn(md, ml, device=dev, generator=gen) * torch.exp(-0.001 * torch.arange(ml, device=dev))[None, :]
            w_q, w_k, w_v = [(torch.randn(md, md, device=dev, generator=gen) / md ** 0.5).to(torch.bfloat16) for _ in range(3)]
            mws = torch.zeros(chela.mixer_workspace_bytes(mb, ml, md, mh, mc), dtype=torch.uint8, device=dev)
            mo = torch.empty(mb, ml, md, device=dev)
            spec = chela.longconv_prepare(k_l)   # the long kernels' spectra, once: the weights do not change between calls
            ms = timed(lambda: chela.mixer_prepared_fwd(x, w_s, spec, w_q, w_k, w_v, mh, chunk=mc, out=mo, workspace=mws), 20, warm=5)
            mhz_mixer = chela.debug_sm_clock_mhz()
            ms_unprepared = timed(lambda: chela.mixer_fwd(x, w_s, k_l, w_q, w_k, w_v, mh, chunk=mc, out=mo, workspace=mws), 10, warm=3)
            if chela.async_status(mws) != chela.OK:
                raise RuntimeError("device-side wait timed out in the mixer")
            d_head = md // mh
            flops_tok = mixer_flops_per_token(md, mh)
            mixers.append({"B": mb, "L": ml, "D": md, "H": mh, "chunk": mc, "attention_tile_tokens": 64, "ms": ms, "sm_mhz_counted": mhz_mixer, "ms_spectra_recomputed_every_call": ms_unprepared,
                           "call": "chela_mixer_prepared_fwd (kernel spectra prepared once with chela_longconv_prepare)",
                           "tokens_per_s": mb * ml / (ms * 1e-3),
                           "tensor_frac": flops_tok * mb * ml / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                           "attention_kernel_kind": chela.linattn_kernel_kind(mb, mh, ml, d_head, d_head, mc,
                                                                              chela.BF16_PAIR)})
            # the prologue stages and one projection of the same shapes on their own (rows a1, a2, a3 of the path)
            stage = {}
            y_s = torch.empty_like(x)
            ms_s = timed(lambda: chela.shortconv_fwd(x, w_s, out=y_s), 20, warm=5)
            stage["shortconv"] = {"ms": ms_s, "GBps": 2 * x.numel() * 2 / (ms_s * 1e-3) / 1e9,
                                  "hbm_frac": 2 * x.numel() * 2 / (ms_s * 1e-3) / 1e9 / peaks["hbm_gbs"]}
            z_l = torch.empty(mb, ml, md, device=dev)
            cws = torch.zeros(chela.longconv_workspace_bytes(mb, ml, md, chela.BF16, chela.F32), dtype=torch.uint8, device=dev)
            ms_l = timed(lambda: chela.longconv_fwd(x, k_l, w_s, out=z_l, workspace=cws), 20, warm=5)
            m_pts = 1 << (ml - 1).bit_length()
            fft_flops = (mb * md * 2 + md) * 5 * m_pts * (m_pts.bit_length() - 1)   # forward + inverse per row, forward per kernel
            stage["longconv"] = {"ms": ms_l, "fft_TFLOPs": fft_flops / (ms_l * 1e-3) / 1e12, "alu_peak_TFLOPs": fp32_peak,
                                 "alu_frac": fft_flops / (ms_l * 1e-3) / 1e12 / fp32_peak,
                                 "alu_peak_source": "measured in this run: fp32 GEMM 8192^3 with TF32 off (plain FMA pipes)",
                                 "note": "short conv + SiLU + transposes + FFT long conv, bf16 in, fp32 out; flops = 5 M log2 M "
                                         "per M-point transform"}
            z_p = torch.randn(2, mb * ml, md, device=dev, generator=gen).to(torch.bfloat16)
            q_p = torch.empty(2, mb * ml, md, device=dev, dtype=torch.bfloat16)
            dws = torch.zeros(max(int(chela.lib().chela_dense_workspace_bytes()), 16), dtype=torch.uint8, device=dev)
            ms_d = timed(lambda: chela.dense_fwd(z_p, w_q, a_dtype=chela.BF16_PAIR, y_dtype=chela.BF16_PAIR, out=q_p, workspace=dws), 20, warm=5)
            mma_flops = 2 * 2.0 * mb * ml * md * md   # two tensor-core terms per product (pair operand)
            stage["projection"] = {"ms": ms_d, "TFLOPs": mma_flops / (ms_d * 1e-3) / 1e12,
                                   "tensor_frac": mma_flops / (ms_d * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                   "note": "one Q or K projection, bf16-pair A (token-major) and Y: both tensor-core terms counted"}
            mixers[-1]["stages"] = stage
            # the gated form (Eqs. 8-14): two more projections and the gate epilogue
            w_a, w_o2 = [(torch.randn(md, md, device=dev, generator=gen) / md ** 0.5).to(torch.bfloat16) for _ in range(2)]
            gws = torch.zeros(chela.mixer_gated_workspace_bytes(mb, ml, md, mh, mc), dtype=torch.uint8, device=dev)
            ms_gt = timed(lambda: chela.mixer_prepared_fwd(x, w_s, spec, w_q, w_k, w_v, mh, w_a=w_a, w_o=w_o2, chunk=mc, out=mo, workspace=gws), 10, warm=3)
            if chela.async_status(gws) != chela.OK:
                raise RuntimeError("device-side wait timed out in the gated mixer")
            mixers[-1]["gated"] = {"ms": ms_gt, "tokens_per_s": mb * ml / (ms_gt * 1e-3),
                                   "tensor_frac": mixer_flops_per_token(md, mh, True) * mb * ml / (ms_gt * 1e-3) / 1e12 / peaks["bf16_tflops"]}
            del gws, w_a, w_o2
            del x, k_l, mws, mo, y_s, z_l, cws, z_p, q_p, dws, spec
        line["mixer"] = mixers
        # ---- backward of the timed workload (gradients w.r.t. Q, K, V; normaliser on) ----------------------------
        (q_, k_, v_), _ = views(L_MAIN)
        d_o = (torch.randn(q_.shape, device=dev, generator=gen)).to(torch.bfloat16)
        bws = torch.zeros(int(chela.lib().chela_linattn_bwd_workspace_bytes(q_.shape[0], H, L_MAIN, D, D)), dtype=torch.uint8, device=dev)
        ms = timed(lambda: chela.linattn_bwd(q_, k_, v_, d_o, workspace=bws), 10, warm=3)
        mhz_bwd = chela.debug_sm_clock_mhz()
        if chela.async_status(bws) != chela.OK:
            raise RuntimeError("device-side wait timed out in the backward pass")
        bwd_alg = TOTAL_TOKENS * H * D * (4 * 2 + 3 * 4)   # read q, k, v, d_o (bf16), write dq, dk, dv (fp32): 20 B per element
        line["backward"] = {"ms": ms, "sm_mhz_counted": mhz_bwd, "tokens_per_s": TOTAL_TOKENS / (ms * 1e-3),
                            "roofline": {"bound": "hbm", "achieved": bwd_alg / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                         "frac": bwd_alg / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None, "peak_source": peak_kind,
                                         "algorithmic_bytes_per_call": bwd_alg},
                            "note": "chela_linattn_bwd, bf16 in, fp32 gradients, same workload as the timed step; algorithmic "
                                    "bytes of a one-pass backward (20 B per element) over the time of the whole multi-launch call"}
        # forward + backward at every L of the sweep (the quantity the paper's runtime-vs-length figure plots)
        fb = []
        sweep_ms = {e["L"]: e["ms"] for e in sweep}
        for L in SWEEP_L:
            (q_, k_, v_), _ = views(L)
            g_ = d_o.view(q_.shape)
            need = int(chela.lib().chela_linattn_bwd_workspace_bytes(q_.shape[0], H, L, D, D))
            if need > bws.numel():
                bws = torch.zeros(need, dtype=torch.uint8, device=dev)
            ms_b = timed(lambda: chela.linattn_bwd(q_, k_, v_, g_, workspace=bws), 5, warm=2)
            if chela.async_status(bws) != chela.OK:
                raise RuntimeError("device-side wait timed out in the backward sweep")
            fb.append({"L": L, "fwd_ms": sweep_ms[L], "bwd_ms": ms_b, "fwd_bwd_ms": sweep_ms[L] + ms_b})
        line["fwd_bwd_sweep"] = fb
        del d_o, bws
        # ---- decode step: one token per sequence against the carried state (bound by the state's bytes) --------
        db, dh = 256, H
        qs, ks, vs = ((torch.randn((db, dh, D), device=dev, generator=gen) * 0.125).to(torch.bfloat16) for _ in range(3))
        states = [torch.zeros((db, dh, D, D), device=dev) for _ in range(3)]   # 3 x 67 MB: rotated, larger than L2
        o_step = torch.empty((db, dh, D), device=dev)
        it = [0]

        def step_once():
            chela.linattn_step(qs, ks, vs, states[it[0] % 3], out=o_step)
            it[0] += 1
        ms = timed(step_once, 30, warm=6)
        line["decode_step"] = {"ms": ms, "sequences": db * dh, "tokens_per_s": db / (ms * 1e-3),
                               "state_GBps": 2 * db * dh * D * D * 4 / (ms * 1e-3) / 1e9,
                               "hbm_frac": 2 * db * dh * D * D * 4 / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                               "note": "chela_linattn_step, B=256 H=16 d=64, fp32 state read and written once per token"}
        del qs, ks, vs, states, o_step
        # ---- CPU oracle on the host cores, bounded sample -----------------------------------------------
        import oracle
        oracle.build()
        nb = max(1, min(4, TOTAL_TOKENS // L_MAIN))
        data = oracle_inputs(nb, L_MAIN)
        time_oracle_sample(oracle_inputs(1, 2048))  # warm the thread pool
        tps, secs, passes, cores = time_oracle_sample(data, budget_s=12.0)
        line["cpu_baseline"] = {"value": tps, "unit": "tokens/s", "cores": cores, "kind": "oracle", "seconds": secs,
                                "sample": "recurrent-form float64 oracle, %d passes over %d of the %d batch rows of the "
                                          "step (B=%d, L=%d, H=16, d=64)" % (passes, nb, TOTAL_TOKENS // L_MAIN, nb, L_MAIN)}
    sampler.stop()
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
