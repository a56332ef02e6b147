"""world_size 2 over gloo on CPU: what the ranks of one GVA space exchange on the host.  Each rank owns a pool
(the oracle stands in for the device library here: no GPU), exports its mapping and its ready samples'
descriptors, all-gathers them, and then every rank computes the same plan redundantly (Algorithm 1 is
deterministic) and takes the microbatches the zig-zag dealt to it."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import hashlib, json, os, sys
sys.path.insert(0, {root!r}); sys.path.insert(0, os.path.join({root!r}, "tests"))
import numpy as np, torch.distributed as dist
import workloads
from harness import pool_config_fields, plan_config_fields, register_args, write_args, host_span
from oracle import OraclePool, PoolConfig, PlanConfig, plan_from_lengths
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = workloads.make_workload("image_mix_7b", n_samples=12, hidden=56, page_bytes=4096)
w.n_ranks_N = world
f = pool_config_fields(w); f.update(world_size=world, rank=rank)
pool = OraclePool(PoolConfig(**f)); assert pool.rc == 0
mine = [s for s in range(w.n_samples) if s % world == rank]          # each producer writes its own samples
assert pool.register_samples(*register_args(w, mine)) == 0
call = [(s, j) for s in mine for j in range(int(w.n_spans[s]))]
assert pool.write_embeddings(*write_args(w, call), [host_span(w, s, j) for s, j in call], 0) == 0
# exchange: mapping blobs once, then (slot, length) of the ready samples
maps = [None] * world
dist.all_gather_object(maps, pool.export_mapping()[1].tobytes())
meta = [None] * world
dist.all_gather_object(meta, [(int(s), int(w.seq_len[s])) for s in mine])
# a peer's mapping blob parses and names its rank; own blob is refused (another process's frames cannot be reached
# from this CPU process, so the import itself is exercised with a null peer and must say INVALID_ARG)
for r in range(world):
    blob = np.frombuffer(maps[r], dtype=np.uint8)
    assert pool.import_mapping(blob, None) == -1
# the same global list on every rank -> the same plan on every rank
glob = sorted(x for part in meta for x in part)
slots = [s for s, _ in glob]; lens = [l for _, l in glob]
rc, plan = plan_from_lengths(lens, PlanConfig(**plan_config_fields(w)), slots=slots)
assert rc == 0
a = plan.arrays()
digest = hashlib.sha256(b"".join(np.ascontiguousarray(a[k]).tobytes() for k in sorted(a) if k != "n_mb")).hexdigest()
digests = [None] * world
dist.all_gather_object(digests, digest)
assert len(set(digests)) == 1
my_mbs = [int(j) for j in a["rank_mbs"][a["rank_mb_off"][rank]:a["rank_mb_off"][rank + 1]]]
taken = [None] * world
dist.all_gather_object(taken, my_mbs)
if rank == 0:
    allmb = sorted(j for part in taken for j in part)
    print(json.dumps({{"n_mb": int(a["n_mb"]), "covered": allmb == list(range(int(a["n_mb"]))), "per_rank": [len(t) for t in taken]}}))
dist.barrier(); dist.destroy_process_group()
"""


def test_two_ranks_exchange_descriptors_and_plan_identically(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29541", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=600) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["covered"] and line["n_mb"] >= 2
    assert abs(line["per_rank"][0] - line["per_rank"][1]) <= 4     # one bucket at most one apart, four buckets
