"""Host-side logic of bench.py: flop accounting, the reference arm's JSON line and
the multi-rank plumbing (world size 2 over gloo on the CPU)."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_flop_accounting():
    f_ap, f_e2e = bench.step_flops()
    per_block = 202_375_168
    assert f_ap == 3 * 2 * 4096 * per_block          # 4.97 TFLOP per block and mode at 4096 tokens
    assert f_e2e == 3 * 2 * 16384 * per_block        # 19.89 TFLOP at 16384 tokens
    assert round(f_ap / 1e12, 2) == 4.97 and round(f_e2e / 1e12, 2) == 19.89


def test_peaks_have_a_source():
    p = bench.load_peaks()
    assert p["source"] in ("measured", "fallback")
    assert p["hbm_gbs"] > 1000 and p["bf16_tflops_sustained"] > 100


def test_traffic_figures_follow_the_kernel_sources(monkeypatch):
    """The ncu DRAM figures are reported only for the kernel sources they were captured from."""
    t = bench.traffic_per_launch("packed_fwd")
    if t is None:
        pytest.skip("gemm.cu or ptx.cuh changed since the last ncu capture (bench.py then reports traffic: null)")
    table = bench.NCU_TRAFFIC["packed_fwd"]
    assert t == pytest.approx((4 * table["qkvo"] + 2 * table["gate_up"] + table["down"]) / 7)
    assert 0.5 < t / 372.7e6 < 1.5                       # near the algorithmic bytes of a forward launch
    assert bench.traffic_per_launch("fakequant_fwd") is None
    monkeypatch.setitem(bench.NCU_TRAFFIC, "sources_sha256", "0" * 64)
    assert bench.traffic_per_launch("packed_fwd") is None


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, rank, world)
        bench.barrier()
        slowest = bench.max_over_ranks(10.0 + rank, torch.device("cpu"))
        q.put((rank, slowest))
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_world2_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 11.0), (1, 11.0)]             # every rank sees the slowest rank's time


def test_reference_arm_line_and_idle_ranks():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, env=env, timeout=600)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"] == bench.WORKLOAD
    assert line["cpu_baseline"]["cores"] >= 1 and line["cpu_baseline"]["threads"]["element-wise steps, group sums, bit packing"] == 1
    assert 0.0 < line["cpu_baseline"]["time_share_of_matrix_products"] < 1.0
    # under torchrun only rank 0 works; the others exit 0 silently
    env1 = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out1 = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                           "--warmup", "0", "--gpus", "2"], capture_output=True, text=True, env=env1, timeout=600)
    assert out1.returncode == 0 and out1.stdout.strip() == ""


def test_gpus_flag_spawns_the_ranks_itself():
    """`bench.py --gpus 2` with no launcher around it starts two ranks (here on the CPU, through the reference arm):
    exactly one line comes back, rank 0's, and it says n_gpus 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--gpus", "2"], capture_output=True, text=True, env=env, timeout=600)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2


def test_rooflines_carry_every_denominator():
    peaks = bench.load_peaks()
    r = bench.tensor_roofline(1000.0, peaks, 0.4, 1500.0)
    assert r["peak"] == peaks["bf16_tflops"] and "burst" in r["peak_source"]            # a short timed region
    assert r["frac_vs_burst"] == pytest.approx(1000.0 / peaks["bf16_tflops"])
    assert r["frac_vs_sustained"] == pytest.approx(1000.0 / peaks["bf16_tflops_sustained"])
    assert r["frac_vs_nominal"] == pytest.approx(1000.0 / 2250.0)
    assert bench.tensor_roofline(1000.0, peaks, 5.0, 1400.0)["peak"] == peaks["bf16_tflops_sustained"]
    h = bench.hbm_roofline(4000.0, peaks)
    assert h["frac"] == pytest.approx(4000.0 / peaks["hbm_gbs"]) and h["frac_vs_nominal"] == pytest.approx(0.5)


def test_extra_configs_match_the_workload_table():
    from workloads import CONFIGS
    by_name = {c.name: c for c in CONFIGS}
    for name, spec in bench.EXTRA_CONFIGS.items():
        c = by_name[name]
        assert (spec["bits"], spec["group"]) == (c.bits, c.group)
        assert c.linears == bench.LINEARS[spec["model"]]
        assert {spec["t_ap"], spec["t_e2e"]} - {0} == {c.tokens}
        assert (spec["t_ap"] > 0) == ("block_ap" in c.modes) and (spec["t_e2e"] > 0) == ("e2e_qp" in c.modes)
        assert spec["w"] == (c.weight_dist, c.weight_scale, c.outlier_frac)
