"""Host-side logic of bench.py that needs no GPU: the N > 1 aggregation (replicas only: no data-path collective,
time = max over ranks, value = sum of the replicas' work / that time) on a world-size-2 gloo group, and the
clock-sample parser."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    bench.barrier(world)
    local_ms = 0.100 if rank == 0 else 0.125          # rank 1 is the slow replica
    ms = bench.max_over_ranks(local_ms, world)
    out[rank] = (ms, bench.whole_job_value(ms, world))
    bench.barrier(world)
    dist.destroy_process_group()


def test_replica_aggregation_world_size_2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
    import bench

    assert out[0] == out[1]
    ms, value = out[0]
    assert ms == pytest.approx(0.125)
    assert value == pytest.approx(2 * bench.retained_flops(0.5) / 0.125e-3 / 1e12)
    assert bench.whole_job_value(0.125, 1) == pytest.approx(value / 2)


def test_retained_flops_and_single_rank():
    import bench

    assert bench.retained_flops(0.5) == 2.0 * 32768 * 14336 * 8192          # the headline: 70B-class down projection
    assert bench.retained_flops(1.0) == 2.0 * 32768 * 28672 * 8192
    assert bench.retained_flops(0.5, 2048, 8192, 2048) == 2.0 * 2048 * 4096 * 2048
    assert bench.max_over_ranks(1.5, 1) == 1.5


def test_roofline_denominator_follows_the_sampled_clocks():
    """The GEMM's roofline fraction is taken against the sustained cuBLAS rate only when the SM clock sampled during
    the timed region sagged, against the burst rate otherwise; recomputing achieved / peak gives the reported fraction."""
    import bench

    peaks = {"bf16_burst": 1600.0, "bf16_sustained": 1300.0, "hbm_gbs": 6500.0, "source": "measured"}
    hot = bench.gemm_roofline(1000.0, 5.0, peaks, {"sm_mhz": 1300.0, "sm_max_mhz": 1965.0}, None)
    cool = bench.gemm_roofline(1000.0, 0.03, peaks, {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0}, 1e6)
    assert hot["peak"] == 1300.0 and cool["peak"] == 1600.0
    for r in (hot, cool):
        assert r["frac"] == pytest.approx(r["achieved"] / r["peak"])
        assert r["frac_of_nominal_peak"] == pytest.approx(1000.0 / 2250.0)
    assert bench.gemm_roofline(1000.0, 1.0, peaks, {"sm_mhz": None, "sm_max_mhz": None}, None)["peak"] == 1600.0


def test_clock_sample_parser():
    import bench

    s = bench.ClockSampler(0)
    s.proc = object()
    s.lines = ["1965, 1965, 310.5, 0x0000000000000000, Not Active, Not Active, Not Active, Not Active",
               "1320, 1965, 995.0, 0x0000000000000004, Not Active, Not Active, Not Active, Active",
               "1305, 1965, 996.0, 0x0000000000000004, Not Active, Not Active, Not Active, Active", "garbage"]

    class P:
        def terminate(self): pass
        def wait(self, timeout=None): pass
    s.proc = P()
    r = s.stop()
    assert r["sm_mhz"] == 1320 and r["sm_max_mhz"] == 1965 and r["reasons"] == ["sw_power_cap"] and r["samples"] == 3
