"""CPU tests of bench.py's host-side logic: the world-size-2 aggregation (gloo), the algorithmic
counts behind the roofline, and the reference (oracle) arm's JSON line."""
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


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r took (10 + 5 r) ms for 1000 (r + 1) units: job time = slowest rank, job units = sum
        ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 1000 * (rank + 1))
        out[rank] = (ms, units)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_aggregate_over_ranks_gloo_world_size_2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29611, out), nprocs=2, join=True)
    assert out[0] == out[1] == (15.0, 3000)


def test_aggregate_without_process_group_is_identity():
    assert bench.aggregate_over_ranks(3.5, 42) == (3.5, 42)


def test_algorithmic_counts():
    assert bench.key_flops_per_vector(128, 1) == 2 * 8128
    assert bench.key_flops_per_vector(128, 32) == 2 * 6144
    assert bench.key_flops_per_vector(128, 64) == 2 * 4096
    assert bench.key_flops_per_vector(128, 1, 32) == 2 * 8128          # r = 32: the triangle (8128) beats 2 r d = 8192
    assert bench.key_flops_per_vector(128, 1, 8) == 2 * 2048           # r = 8: the rank-r form is the cheaper count
    assert bench.key_fma_split(128, 1) == (4 * 496, 8128 - 4 * 496)      # four 32 x 32 triangles stay on the FP32 pipes
    assert sum(bench.key_fma_split(128, 32)) == 6144 and bench.key_fma_split(128, 32)[0] == 0
    assert sum(bench.key_fma_split(128, 64)) == 4096
    assert bench.bytes_per_vector(128, 2, 32, 2) == 320
    assert bench.bytes_per_vector(128, 4, 128, 2) == 328
    assert bench.bytes_per_vector(128, 2, 32, 2, meta_bytes=2) == 304      # binary16 scale and zero
    assert abs(bench.ALU_PEAK_TFLOPS - 74.45) < 0.01
    # the reader: 32 + 32 code bytes, 32 bytes of key metadata, 32 of value metadata per cached token at 2 bits, G = 32
    assert bench.reader_bytes_per_cached_token(128, 2, 32) == 128
    assert bench.reader_bytes_per_cached_token(128, 4, 128) == 64 + 64 + 8 + 8
    assert bench.reader_bytes_per_cached_token(128, 2, 32, meta_bytes=2) == 32 + 32 + 16 + 16


def test_key_roofline_is_the_slowest_of_the_three_floors():
    import argparse
    import squat_inputs as si
    args = argparse.Namespace(meta16=False)
    peaks = {"hbm_gbs": 6549.8, "bf16_tflops": 1649.9, "source": "measured"}
    fp32 = {"tflops": 73.0, "fma_f32_tflops": 71.0, "fma_f32x2_tflops": 73.0}
    cfg = si.get_config(1)
    vec = cfg.batch * cfg.n_kv_heads * cfg.n_tokens
    r = bench.key_roofline(args, cfg, 0.053, vec, peaks, fp32)
    # dense kernel on workload 1: the in-block triangles (1 984 multiply-adds per vector on the FP32 pipes) set the floor
    assert r["bound"] == "alu" and r["peak"] == 73.0
    assert abs(r["pipes"]["fp32_floor_us"] - 2 * 1984 * vec / 73.0e12 * 1e6) < 1e-9
    assert abs(r["pipes"]["tensor_floor_us"] - 6 * 6144 * vec / (0.5 * 1649.9e12) * 1e6) < 1e-9
    assert abs(r["pipes"]["hbm_floor_us"] - 320 * vec / 6549.8e9 * 1e6) < 1e-9
    assert r["pipes"]["floor_us"] == max(r["pipes"][k] for k in ("fp32_floor_us", "tensor_floor_us", "hbm_floor_us"))
    assert abs(r["frac"] - r["pipes"]["floor_us"] / 53.0) < 1e-9 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-12
    assert abs(r["frac_vs_fp32_target"] - 16256 * vec / 0.053e-3 / 1e12 / bench.ALU_PEAK_TFLOPS) < 1e-9
    # the rank-r kernel runs 2 r d multiply-adds per vector on the FP32 pipes and nothing on the tensor cores
    c4 = si.get_config(4).with_(rank_r=8)
    r8 = bench.key_roofline(args, c4, 1.0, 4 * 32 * 32768, peaks, fp32, lowrank_r=8)
    assert r8["pipes"]["fp32_fma_per_vector"] == 2048 and r8["pipes"]["tensor_fma_per_vector"] == 0
    assert r8["bound"] in ("alu", "hbm") and r8["kernel"].startswith("quant_keys_lowrank_kernel")
    # W = 0: nothing to push, the bytes bind
    r0 = bench.key_roofline(args, cfg.with_(rank_r=0), 0.05, vec, peaks, fp32)
    assert r0["bound"] == "hbm"


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "key_vectors/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    env["RANK"], env["WORLD_SIZE"] = "1", "2"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0"],
                       capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0 and r.stdout.strip() == ""
