"""Host-side logic of bench.py without a GPU: multi-rank aggregation under gloo (world size 2), the
reference arm's JSON line, and the clock-sampler summary."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    out[rank] = (ms, bench.job_tokens_per_s(ms, world, 1000))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_sum_the_work():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, 29513, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, tps = res[0]
    assert ms == 15.0
    assert abs(tps - 2 * 1000 / 15e-3) < 1e-6


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.job_tokens_per_s(2.0, 1, 262144) == 262144 / 2e-3


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "1", "--tokens", "4096", "--L", "1024"], capture_output=True, text=True, env=env,
                         timeout=600, check=True).stdout.strip().splitlines()
    line = json.loads(out[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["vs_baseline"] is None


def test_clock_sampler_summary_window():
    s = bench.ClockSampler.__new__(bench.ClockSampler)

    class FakeNvml:
        nvmlClocksEventReasonSwPowerCap = 0x4
        nvmlClocksEventReasonHwSlowdown = 0x8
        nvmlClocksEventReasonSwThermalSlowdown = 0x20
        nvmlClocksEventReasonHwThermalSlowdown = 0x40
        nvmlClocksEventReasonHwPowerBrakeSlowdown = 0x80

    s.nv, s.max_mhz = FakeNvml, 1965
    s.samples = [(0.5, 1000, 0), (1.1, 1900, 0x4), (1.2, 1950, 0x4), (1.3, 1965, 0), (2.5, 500, 0x8)]
    got = s.summary(1.0, 2.0)
    assert got == {"sm_mhz": 1950, "sm_max_mhz": 1965, "reasons": ["sw_power_cap"], "samples": 3}
