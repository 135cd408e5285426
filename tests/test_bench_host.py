"""Host-side logic of bench.py: algorithmic byte counts, the reference arm's JSON line, and the
multi-rank reduction (world size 2 over gloo on CPU; ranks are independent replicas)."""
import json
import os
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from synth import CONFIGS  # noqa: E402


def test_algorithmic_bytes_count_every_byte_once():
    # Per image at the 2880-token shape: attention rows 0.18 MB + head means and kept list 0.02 MB, features
    # once and merged rows out 6.55 MB, keys of the visual span 2.63 MB, and the compaction's 12.73 MB of rows
    # read and written less the 1.31 MB of surviving key rows that the scoring has already read: 20.8 MB.
    a2, a1 = bench.algorithmic_bytes(CONFIGS[2]), bench.algorithmic_bytes(CONFIGS[1])
    assert abs(a2["step"] / 32 / 1e6 - 20.82) < 0.05
    assert abs(a2["compact"] / 32 / 1e6 - (12.73 - 1.31)) < 0.02
    assert abs(a2["qk_softmax"] / 32 / 1e6 - 2.63) < 0.01
    assert a2["step"] == a2["score_select"] + a2["merge"] + a2["prune_fused"]
    e, c = 2, CONFIGS[2]
    survivors = c.B * c.Hkv * c.k2 * c.d * e
    rows_moved = c.B * 2 * c.S_out * (c.Dh * e + 2 * c.Hkv * c.d * e + 4)
    assert a2["compact"] == rows_moved - survivors
    assert abs(a1["compact"] / 256 / 1e6 - (9.59 - 0.79)) < 0.02
    assert abs(bench.merge_flops(CONFIGS[2]) / 160 / 1e6 - 67.1) < 0.1
    assert abs(bench.merge_flops(CONFIGS[3]) / 4 / 1e9 - 75.2) < 0.1


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port), VSCAN_BENCH_BACKEND="gloo")
    r, w, lr, dist = bench.dist_setup(world)
    assert (r, w, lr) == (rank, world, rank)
    dist.barrier()
    out[rank] = bench.max_over_ranks(10.0 + 5 * rank, dist, torch.device("cpu"))
    dist.destroy_process_group()


def test_max_over_ranks_gloo_world2():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29517, out), nprocs=2, join=True)
    assert out[0] == out[1] == 15.0
    assert bench.max_over_ranks(3.5, None, None) == 3.5


def test_reference_arm_prints_contract_line():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1"], capture_output=True, text=True, check=True, cwd=ROOT)
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "images/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["steps"] == 2
    # under torchrun only rank 0 works; the other ranks exit 0 silently
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, check=True, cwd=ROOT,
                         env=env)
    assert res.stdout.strip() == ""
