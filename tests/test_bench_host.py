"""Host-side logic of bench.py: byte/flop accounting against hand-computed figures, and the N > 1 path
(max over ranks, weak-scaling aggregation) on two gloo ranks."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_weight_and_kv_bytes_match_hand_computed_totals():
    cfg = synth.get_config("latency_8b")
    a = bench.workload_accounting(cfg, [2048], 1, 16)
    # 8B-class: Proj_dS alone is 4096 x 1 048 576 x 2 B = 8.59 GB; all GEMM weights 10.97 GB
    assert cfg["d_S"] == 1048576
    assert abs(a["weight_bytes"] / 1e9 - 10.97) < 0.02
    # target KV: 4 KiB per token per attention layer, 2 layers
    assert a["kv_bytes"] == 2048 * 4096 * 2
    assert a["drafter_kv_bytes_avoided"] == a["kv_bytes"]
    cfg = synth.get_config("conc128_32b")
    a = bench.workload_accounting(cfg, [1000] * 128, 128, 16)
    assert abs(a["weight_bytes"] / 1e9 - 17.64) < 0.03
    # dense flops: 2 * rows * params with rows = B for the two state projections, B*k elsewhere
    per_layer = (21664 * 5120 + 5120 * 10240 + 10240 * 5120 + 5120 * 8192 + 51200 * 5120 + 5120 * 25600)
    expect = 2 * 2048 * (2 * per_layer + 152064 * 5120) + 2 * 128 * (5120 * 5120 + 1310720 * 5120)
    assert a["gemm_flops"] == pytest.approx(expect, rel=1e-12)
    # a window limits the visible prefix
    a_w = bench.workload_accounting(dict(cfg, window=513), [1000] * 128, 128, 16)
    assert a_w["kv_bytes"] == 128 * 512 * 4096 * 2


def test_peaks_fallback_and_file(tmp_path, monkeypatch):
    p = bench.load_peaks()
    assert p["hbm_gbs"] > 1000 and p["bf16_tflops_sustained"] > 100 and p["source"] in ("measured", "fallback")


def test_serial_roofline_sums_each_launch_at_its_own_bound():
    peaks = dict(hbm_gbs=1000.0, bf16_tflops_sustained=100.0)
    launches = [("gemm:proj_ds", 1e9, 2e9),          # streaming: 2 GB at 1 TB/s = 2 ms (its flops would take 0.01 ms)
                ("gemm2:gate_up", 4e11, 1e8),        # tensor-bound: 4e11 flops at 100 TF/s = 4 ms (bytes 0.1 ms)
                ("mamba_scan", 1e6, 5e8),            # 0.5 ms of state bytes
                ("rmsnorm", 0.0, 9e9)]               # row-wise kernels are not counted
    assert bench.serial_roofline_ms(launches, 1e9, peaks) == pytest.approx(2.0 + 4.0 + 0.5 + 1.0)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_info()[0] == rank and bench.dist_info()[2] == world
        bench.barrier()
        slow = bench.max_over_ranks(10.0 + 5.0 * rank)           # rank 1 is the slow one
        units = 128 * 16 * world                                  # weak scaling: every rank drafts its own batch
        out[rank] = (slow, units / (slow * 1e-3))
    finally:
        dist.destroy_process_group()


def test_two_rank_replicas_take_the_max_time():
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0][0] == 15.0 and out[1][0] == 15.0               # every rank sees the slowest rank's time
    assert out[0][1] == pytest.approx(2 * 128 * 16 / 15e-3)


def test_reference_arm_prints_one_contract_line_on_cpu():
    """`bench.py --impl reference` times the oracle on the host cores and prints one JSON line with the contract's keys
    (run here on the tiny workload; no GPU involved)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["higher_is_better"] is True
    for key in ("metric", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "scaling", "vs_baseline", "dtype", "data",
                "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"] == "tiny"
