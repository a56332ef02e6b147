"""The launch-geometry knobs (pool_set_tuning) change how the copy kernels are launched, never what they compute:
the same two-tier workloads, written and assembled under unusual settings, must equal the oracle bit for bit."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import workloads
from test_gpu_parity import assert_same, oracle_from_device_sources

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

TUNINGS = [
    dict(dev_ctas_per_sm=1, scatter_ctas_per_sm=1, gather_unroll=8),
    dict(dev_ctas_per_sm=8, scatter_ctas_per_sm=8, scatter_group=5, chunk_shift=14),
    dict(chunk_shift=21, host_ctas=1, host_store_ctas=1, scatter_smem_carveout=30, gather_smem_carveout=30),
    dict(host_ctas=13, host_store_ctas=17, scatter_group=2, chunk_shift=18),
    dict(host_copy_engine=1),                      # host-tier pages by cudaMemcpyAsync runs instead of the bulk-copy kernels
    dict(host_copy_engine=1, chunk_shift=14, dev_ctas_per_sm=2),
]


@pytest.mark.parametrize("tuning", TUNINGS)
@pytest.mark.parametrize("name,kw", [
    ("image_mix_7b", dict(n_samples=10, hidden=512, page_bytes=65536)),      # both tiers, rows straddle pages
    ("host_tier_stress", dict(n_samples=4, hidden=1024, page_bytes=16384)),  # fp32 source, tiers interleaved
])
def test_results_do_not_depend_on_the_launch_geometry(name, kw, tuning):
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import run_cuda
    w = workloads.make_workload(name, **kw)
    got = run_cuda(w, tuning=tuning)
    exp = oracle_from_device_sources(w, got["srcs"], got["table"])
    assert_same(got, exp)
    assert not np.any(np.all(got["out"] == 0xFFFF, axis=1))


@pytest.mark.parametrize("name,kw", [
    ("image_mix_7b", dict(n_samples=10, hidden=512, page_bytes=16384)),     # spans of several pages each
    ("image_mix_7b", dict(n_samples=6)),                                     # 2 MiB pages, 7 KiB rows
])
def test_copy_engine_runs_over_contiguous_host_frames(name, kw):
    """With an identity binding and the sorted ring, the host-tier pages of a span are consecutive frames, so the
    copy-engine path merges them into one copy per run (with the permuted binding of the other cases every run is
    one page).  Written and assembled that way, the result must equal the oracle bit for bit."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import run_cuda
    w = workloads.make_workload(name, **kw)
    w.bind_order = 0
    assert w.ring_order == 0 and w.host_pages > 0
    got = run_cuda(w, tuning=dict(host_copy_engine=1))
    exp = oracle_from_device_sources(w, got["srcs"], got["table"])
    assert_same(got, exp)
    assert not np.any(np.all(got["out"] == 0xFFFF, axis=1))


def test_tuning_round_trip_and_range_checks():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from harness import pool_config_fields
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("tiny")
    pool = fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    d = pool.get_tuning()
    assert (d["dev_ctas_per_sm"], d["scatter_ctas_per_sm"], d["chunk_shift"], d["host_ctas"], d["gather_unroll"]) == (0, 4, 0, 6, 0)   # 0: chosen per call or per launch
    assert d["scatter_smem_carveout"] == 5 and d["gather_smem_carveout"] == 0 and d["remote_ctas"] == 16
    for bad in (dict(chunk_shift=13), dict(chunk_shift=22), dict(gather_unroll=6), dict(dev_ctas_per_sm=9), dict(peers_remote=2),
                dict(scatter_smem_carveout=101), dict(host_copy_engine=3)):
        assert pool.set_tuning(**bad) == -1 and pool.get_tuning() == d          # INVALID_ARG, nothing changed
    assert pool.set_tuning(host_ctas=3, chunk_shift=17) == 0
    t = pool.get_tuning()
    assert t["host_ctas"] == 3 and t["chunk_shift"] == 17 and t["dev_ctas_per_sm"] == 0   # unnamed knobs go back to their defaults
    assert pool.set_tuning() == 0 and pool.get_tuning() == d
    pool.destroy()


def test_a_bulk_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable():
    """The one device-side wait of the library (a bulk-copy CTA waiting for a staged load) is made to run out without
    any fault: under the `bulk_timeout_test` hook every load announces 16 bytes more than it requests, so no load is
    ever seen complete although all of them arrive.  Each host-tier CTA waits 2 ms, gives up, waits once more for the
    loads it had issued, and returns; the call reports FT_ERR_TIMEOUT with the loads it counted as not arrived, stores
    nothing from host frames, and the CUDA context and the pool stay usable: with the hook off, the same plan
    assembles bit-exactly."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import CudaRun, bits16, host_bits
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("image_mix_7b", n_samples=10, hidden=512, page_bytes=65536)
    r = CudaRun(w)
    r.run_schedule()
    assert w.host_pages > 0
    rc, plan = r.plan()
    assert rc == 0
    # the hook is refused without a short limit
    assert r.pool.set_tuning(bulk_timeout_test=1) == -1 and r.pool.set_tuning(bulk_timeout_test=1, bulk_wait_limit_us=200000) == -1
    assert r.pool.set_tuning(bulk_wait_limit_us=50) == -1
    assert r.pool.set_tuning(bulk_timeout_test=1, bulk_wait_limit_us=2000) == 0
    rc, out, cu, pos = r.gather_all()
    assert rc == 0                                           # the error is asynchronous
    code, detail = r.pool.status()
    assert code == -13, fp.STATUS.get(code)                  # FT_ERR_TIMEOUT
    assert (detail >> 16) & 0xFFFF >= 1                      # loads counted as not arrived when the CTA returned
    assert (detail & 0xFFFF) < r.pool.get_tuning()["host_ctas"]
    poisoned = np.all(out.cpu().numpy().view(np.uint16) == 0xFFFF, axis=1)
    assert poisoned.any()                                    # rows that live on host frames were not stored
    assert r.pool.status() == (0, 0)                         # reading clears it
    # a producer call under the hook: same report from the host-tier scatter (into a second pool, to keep this one's data)
    r2 = CudaRun(w, tuning=dict(bulk_timeout_test=1, bulk_wait_limit_us=2000))
    r2.run_schedule()
    torch.cuda.synchronize()
    assert all(c == 0 for c in r2.rc) and r2.pool.status()[0] == -13
    r2.close()
    # hook off: the first pool, its plan and the context still work, bit for bit
    assert r.pool.set_tuning() == 0 and r.pool.get_tuning()["bulk_timeout_test"] == 0
    assert r.pool.get_tuning()["bulk_wait_limit_us"] == 2000000
    rc, out, cu, pos = r.gather_all()
    got = dict(plan=plan.arrays(), rc=r.rc, out=out.cpu().numpy().view(np.uint16), cu_seqlens=cu.cpu().numpy(),
               position_ids=pos.cpu().numpy(), status=r.pool.status(), table=bits16(r.table),
               span_pages={(s, j): r.pool.span_pages(s, j)[1] for call in w.write_calls for s, j in call},
               srcs={c: host_bits(t) for c, t in r.srcs.items()}, stats=r.pool.stats())
    exp = oracle_from_device_sources(w, got["srcs"], got["table"])
    got["rc"] = [c for c in got["rc"]][:len(exp["rc"])]
    assert_same(got, exp)
    r.close()


def test_bench_gpus_2_runs_the_exchange_flow_with_two_ranks_on_this_gpu():
    """`bench.py --gpus 2` launches two ranks by itself; with the gloo backend both may share this GPU (their kernels
    never wait on one another: the ranks meet only in host-side collectives).  One line, from rank 0, with the
    independent-batches value and the exchange flow (every rank writes, all plan alike, each assembles its share from
    everybody's pages) beside it."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["FLOWPOOL_BENCH_BACKEND"] = "gloo"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--samples", "48", "--steps", "1", "--warmup", "3",
                          "--skip-e2e", "--skip-cpu"], capture_output=True, text=True, timeout=900, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [json.loads(l) for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["n_gpus"] == 2 and line["value"] > 0 and line["scaling"] == "weak"
    ex = line["exchange"]
    assert ex["config"]["ranks"] == 2 and len(ex["per_rank"]) == 2 and ex["value"] > 0
    assert sum(r["rows"] for r in ex["per_rank"]) == ex["config"]["packed_tokens_all_ranks"]
    assert all(r["bytes_from_peers"] > 0 and r["gather_gbs"] > 0 for r in ex["per_rank"])
    assert ex["bytes_over_nvlink_per_step"] == 0            # both ranks on one GPU here


def test_a_call_larger_than_the_preallocated_contexts_grows_them():
    """20 000 one-token spans in ONE register call and ONE write call: their descriptors (320 KB) exceed both the
    pinned staging (64 KiB) and the device scratch (256 KiB) every call context starts with, so the contexts grow in
    the middle of the run; page lists and every assembled byte must still equal the oracle's."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import run_cuda
    from workloads.gen import _assemble
    n = 5000
    w = _assemble("many_spans", 9, 64, 4096, np.full(n, 6), [[1, 1, 1, 1]] * n, budget_L=2048)
    w.hbm_pages, w.host_pages = 3 * n, n + 32          # both tiers
    order = list(range(n))
    w.write_calls = [[(s, j) for s in order for j in range(4)]]
    w.plan_order = order
    got = run_cuda(w)
    exp = oracle_from_device_sources(w, got["srcs"], got["table"])
    assert_same(got, exp)
    assert not np.any(np.all(got["out"] == 0xFFFF, axis=1))


def test_a_plan_may_outlive_its_pool_and_plans_may_pile_up():
    """Plan blocks come from a per-pool cache: a dozen plans alive at once, destroyed in another order, and one
    destroyed after its pool is gone."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import CudaRun
    w = workloads.make_workload("tiny")
    run = CudaRun(w)
    run.run_schedule()
    plans = []
    for _ in range(12):
        rc, plan = run.plan()
        assert rc == 0
        plans.append(plan)
    ref = plans[0].arrays()
    for p in plans[1:]:
        a = p.arrays()
        assert all(np.array_equal(a[k], ref[k]) for k in ref)
    for p in plans[3:] + plans[1:3]:
        p.destroy()
    rc, plan = run.plan()                     # takes a cached block
    assert rc == 0
    rc, out, cu, pos = run.gather_all()
    assert rc == 0 and run.pool.status() == (0, 0)
    plan.destroy()
    run.plan_handle = None
    last = plans[0]
    torch.cuda.synchronize()
    run.pool.destroy()
    last.destroy()                            # its pool no longer exists: the block is freed directly
