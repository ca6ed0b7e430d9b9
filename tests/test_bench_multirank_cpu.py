"""The benchmark's multi-rank rule (replicas only: per-rank work, max-over-ranks time, whole-job rate)
exercised with two gloo ranks on CPU; and the reference arm's behaviour on non-zero ranks."""
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 100.0 if rank == 0 else 250.0          # rank 1 is the slow replica
    ms = bench.max_over_ranks(local_ms, dist)
    q.put((rank, ms, bench.whole_job_rate(256, 10, world, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, rate in res:
        assert ms == 250.0                              # the slowest rank decides
        assert abs(rate - 2 * 256 * 10 / 0.25) < 1e-6   # both replicas' units over that time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(12.5) == 12.5
    assert bench.whole_job_rate(256, 4, 1, 100.0) == 256 * 4 / 0.1


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_roofline_fractions_against_denominators_the_kernel_cannot_beat():
    # figures of the kind a run produces: 1560 TFLOP/s achieved at a sampled SM clock of 1627 MHz (maximum 1965)
    import bench
    peaks = dict(hbm_gbs=6448.4, bf16_burst=1654.2, bf16_sustained=1380.5, source="measured")
    r = bench.roofline_entry(1560.3, peaks, dict(sm_mhz=1627.0, sm_max_mhz=1965.0), sm_count=148)
    assert r["peak"] == 1380.5 and abs(r["frac"] - 1560.3 / 1380.5) < 1e-12         # the library GEMM a kernel may beat
    hw_sampled = 148 * 8192 * 1627.0e6 / 1e12
    hw_max = 148 * 8192 * 1965.0e6 / 1e12
    assert abs(r["hw_peak_at_sampled_clock"] - hw_sampled) < 1e-9 and abs(r["hw_peak_at_max_clock"] - hw_max) < 1e-9
    assert abs(r["frac_of_hw_peak_at_sampled_clock"] - 1560.3 / hw_sampled) < 1e-12
    assert r["frac_of_hw_peak_at_max_clock"] < r["frac_of_hw_peak_at_sampled_clock"] <= 1.0
    # the unit-count peak lies above every measured figure it is compared with: the library GEMMs and the nominal 2.25 PFLOP/s
    assert hw_max > 2250.0 > peaks["bf16_burst"] > peaks["bf16_sustained"]
    # without clock samples only the maximum-clock fraction is given; without a measurement, none
    r = bench.roofline_entry(1560.3, peaks, dict(sm_mhz=None, sm_max_mhz=None))
    assert "frac_of_hw_peak_at_sampled_clock" not in r and r["frac_of_hw_peak_at_max_clock"] < 1.0
    assert bench.roofline_entry(None, peaks, {})["frac"] is None


def test_config_object_is_the_same_for_both_arms():
    import bench
    from paper_2502_01703_b200 import workloads as W
    c = bench.bench_config(W.CONFIGS[bench.WORKLOAD])
    assert c["workload"] == "c2_project_quantize" and c["P"] == 1 << 23 and c["d"] == 8192 and c["bits"] == 4
    assert "model" not in c
