"""Host-side logic of bench.py that needs no GPU: byte accounting, the reference arm, and the multi-rank
path (world_size 2 over gloo on CPU): max-over-ranks timing and rank-0-only printing."""
import json
import os
import subprocess
import sys

import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_algorithmic_bytes_are_4h_per_token():
    w = workloads.make_workload("image_mix_7b", n_samples=8)
    wb, gb = bench.algorithmic_bytes(w)
    assert wb == w.total_vision_tokens * 4 * 3584 and gb == w.total_tokens * 4 * 3584
    w4 = workloads.make_workload("host_tier_stress", n_samples=2)
    assert bench.algorithmic_bytes(w4)[0] == w4.total_vision_tokens * 6 * 8192   # fp32 source: 6H per token


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--samples", "4"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, device="cpu")
total = bench.aggregate_value(1000.0, dist.get_world_size(), ms)
if rank == 0:
    print(json.dumps({{"ms": ms, "value": total, "world": dist.get_world_size()}}))
dist.barrier()
dist.destroy_process_group()
"""


def test_two_rank_timing_is_max_over_ranks_and_value_is_whole_job(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29531", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-1500:] for o in outs]
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["world"] == 2 and line["ms"] == 15.0          # the slower rank's time
    assert abs(line["value"] - 2 * 1000.0 / 15.0 / 1e6) < 1e-12  # bytes of both ranks over that time
    assert outs[1][0].strip() == ""                            # only rank 0 prints


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_gpus_n_launches_n_ranks_by_itself():
    """`bench.py --gpus 2` with no torchrun around it must start two ranks (here: the host-side plumbing only, gloo on
    CPU): rendezvous, slot-size agreement, the length-prefixed descriptor all-gather, one line from rank 0."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--host-logic-only"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1                                  # only rank 0 prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["blobs_ok"] is True
    assert lines[0]["ms_per_step"] == 11.0                  # the slower rank's time


def test_world_size_must_match_gpus():
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "8", "--host-logic-only"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode != 0 and "n_gpus" not in out.stdout


def test_blob_exchange_refuses_an_oversized_blob():
    import numpy as np
    import pytest

    class FakeDist:
        def get_world_size(self):
            return 1
    x = bench.BlobExchange(FakeDist(), 16, "cpu")
    with pytest.raises(ValueError):
        x.all_gather(np.zeros(17, np.uint8))
