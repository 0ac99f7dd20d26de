"""CPU-only checks of the benchmark's host logic, including the multi-process path over gloo."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["VITINT_ROOT"])
import torch, torch.distributed as dist
import bench, synth_inputs as si
rank, local, world = bench.dist_env()
dist.init_process_group("gloo")
# each rank times something different; every rank must see the maximum
mine = 10.0 + 5.0 * rank
got = bench.max_over_ranks(mine, world)
# ranks draw disjoint images
cfg = si.VIT_TINY_BLOCK
x = si.activations(cfg, batch=1, first_image=rank)
dist.barrier()
with open(os.path.join(os.environ["VITINT_OUT"], f"rank{rank}.json"), "w") as fh:
    json.dump({"rank": rank, "world": world, "max": got, "x0": float(x[0, 0])}, fh)
dist.destroy_process_group()
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_max_over_ranks_and_image_sharding_with_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, VITINT_ROOT=str(ROOT), VITINT_OUT=str(tmp_path), MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in range(2)]
    assert sorted(r["rank"] for r in recs) == [0, 1]
    assert all(r["world"] == 2 and r["max"] == 15.0 for r in recs)
    assert recs[0]["x0"] != recs[1]["x0"]


def test_single_process_reduction_is_identity_and_op_counts():
    import bench
    import synth_inputs as si
    assert bench.max_over_ranks(3.5, 1) == 3.5
    cfg = si.VIT_BASE_LAYER
    # 372.2 GOP per step at batch 128 (2 ops per multiply-accumulate)
    assert abs(bench.layer_ops(cfg, cfg.batch) / 1e9 - 372.2) < 0.1
    m = si.mac_counts(197, 768, 12, 64, 3072)
    assert m["qkv"] == 197 * 768 * 2304 and m["qk"] == 12 * 197 * 197 * 64 and m["fc2"] == 197 * 3072 * 768


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup",
                          "0", "--ref-images", "1"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TOPS" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["config"]["workload"] == "vit_base_layer_b128"


def test_gpus_flag_must_match_the_ranks_that_were_started():
    """`--gpus N` either starts N ranks itself (no WORLD_SIZE in the environment) or insists that the launcher
    started exactly N: a mismatch is an error before any device is touched, never a silent 1-GPU run."""
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--steps", "1"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode != 0 and "--gpus 2 but 1 rank" in out.stderr
