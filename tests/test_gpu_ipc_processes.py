"""Two real processes on one node, each a producer and a consumer (Sec. 3.2: every process addresses every other
process's segment; Sec. 3.4: the packing rule is deterministic, so every rank can compute the same plan).  Each
process writes its own samples into its own pool and sends the other, over a host channel, its mapping blob, its
samples' descriptors and shareable handles of its slabs; each maps the other's slabs, imports both blobs, plans
ALL samples (the same plan on both sides) and assembles only the microbatches dealt to its own rank, reading the
other process's pages in place.  Neither process's kernels ever wait on the other's.  Both outputs must equal the
oracle's two-pool run."""
import multiprocessing as mp
import queue

import numpy as np
import pytest
import torch

import workloads
from harness import bits16, plan_config_fields, pool_config_fields, register_args, write_args

pytestmark = pytest.mark.gpu

KW = dict(n_samples=14, hidden=512, page_bytes=65536, all_hbm=True)


def _workload():
    w = workloads.make_workload("image_mix_7b", **KW)
    w.budget_L = int(w.seq_len.max()) * 2
    w.n_ranks_N = 2
    return w


def _cfg(w, rank):
    f = pool_config_fields(w, max_samples=w.n_samples)
    f.update(world_size=2, rank=rank, bind_seed=100 + rank, ring_seed=200 + rank, max_imported_pages=w.hbm_pages + w.host_pages)
    return f


def _own(w, rank):
    return [s for s in range(w.n_samples) if s % 2 == rank]


def _grids(w, samples):
    gi = [(s, j, workloads.span_grid(w, s, j)) for s in samples for j in range(int(w.n_spans[s]))]
    gi = [t for t in gi if t[2] is not None]
    return [s for s, _, _ in gi], [j for _, j, _ in gi], [g for _, _, g in gi]


def run_rank(rank, to_peer, from_peer):
    """One process of the pair.  Returns (plan arrays, rows, cu_seqlens, positions) of its own rank's share."""
    from paper_2606_23087_b200 import binding as fp
    torch.cuda.set_device(0)
    w = _workload()
    own, theirs = _own(w, rank), _own(w, 1 - rank)
    st = torch.cuda.current_stream().cuda_stream
    pool = fp.Pool(fp.PoolConfig(**_cfg(w, rank)))
    assert pool.rc == 0
    a = register_args(w, own)          # slot = sample id on both sides, for own and imported samples alike
    ids = torch.from_numpy(a[5]).cuda()
    assert pool.register_samples(*a[:5], ids.data_ptr(), st) == 0
    call = [(s, j) for s in own for j in range(int(w.n_spans[s]))]
    srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]
    assert pool.write_embeddings(*write_args(w, call), [t.data_ptr() for t in srcs], w.src_dtype, st) == 0
    assert pool.set_span_grids(*_grids(w, own), st) == 0
    rc1, mblob = pool.export_mapping()
    rc2, sblob = pool.export_samples(own, st)
    rc3, handles = pool.ipc_export()
    assert rc1 == rc2 == rc3 == 0
    to_peer.put(("blobs", mblob.tobytes(), sblob.tobytes(), handles))
    msg = from_peer.get(timeout=300)
    assert msg[0] == "blobs", msg
    rc, hbm, text = fp.ipc_open(msg[3])
    assert rc == 0 and hbm and text
    assert pool.import_mapping(np.frombuffer(msg[1], np.uint8), hbm, 0, text) == 0
    assert pool.import_samples(theirs, np.frombuffer(msg[2], np.uint8), st) == 0
    order = list(range(w.n_samples))
    rc, plan = pool.plan_microbatches(order, fp.PlanConfig(**plan_config_fields(w)), st)
    assert rc == 0
    pa = plan.arrays()
    mine = [int(j) for j in pa["rank_mbs"][pa["rank_mb_off"][rank]:pa["rank_mb_off"][rank + 1]]]
    rows = int(pa["mb_tokens"][mine].sum())
    n_cu = int(sum(int(pa["mb_sample_off"][j + 1] - pa["mb_sample_off"][j]) + 1 for j in mine))
    table = workloads.embed_table(w, device="cuda")
    out = torch.full((max(rows, 1), w.hidden), -1, dtype=torch.int16, device="cuda")
    cu = torch.full((max(n_cu, 1),), -7, dtype=torch.int32, device="cuda")
    pos = torch.full((max(rows, 1),), -7, dtype=torch.int32, device="cuda")
    assert pool.gather_list(plan, mine, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), st) == 0
    torch.cuda.synchronize()
    assert pool.status() == (0, 0)
    res = ({k: np.asarray(v).copy() for k, v in pa.items() if k != "n_mb"}, out.cpu().numpy().view(np.uint16)[:rows].copy(),
           cu.cpu().numpy()[:n_cu].copy(), pos.cpu().numpy()[:rows].copy())
    # release: imports first, then the mapping of the peer's slabs; own samples only after the peer did the same
    assert pool.free(theirs, st) == 0
    torch.cuda.synchronize()
    plan.destroy()
    assert fp.ipc_close(hbm, text) == 0
    to_peer.put(("released",))
    assert from_peer.get(timeout=300)[0] == "released"
    assert pool.free(own, st) == 0
    torch.cuda.synchronize()
    st_ = pool.stats()
    assert st_["pages_free"] == st_["pages_total"]
    pool.destroy()
    return res


def child_main(to_parent, from_parent, result_q):
    try:
        result_q.put(("ok", run_rank(1, to_parent, from_parent)))
    except BaseException as e:   # report instead of leaving the parent waiting
        result_q.put(("error", repr(e)))
        to_parent.put(("error", repr(e)))
        raise


def test_two_processes_plan_alike_and_assemble_their_own_share():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from oracle import OraclePool, PlanConfig, PoolConfig
    ctx = mp.get_context("spawn")
    p2c, c2p, result_q = ctx.Queue(), ctx.Queue(), ctx.Queue()
    child = ctx.Process(target=child_main, args=(c2p, p2c, result_q), daemon=True)
    child.start()
    try:
        got = {0: run_rank(0, p2c, c2p)}
        try:
            tag, payload = result_q.get(timeout=300)
        except queue.Empty:
            pytest.fail("the second process did not answer")
        assert tag == "ok", payload
        got[1] = payload
        child.join(timeout=60)
        assert child.exitcode == 0
        # the oracle's two pools, in this process
        w = _workload()
        o = {r: OraclePool(PoolConfig(**_cfg(w, r))) for r in (0, 1)}
        for r in (0, 1):
            own = _own(w, r)
            assert o[r].register_samples(*register_args(w, own)) == 0
            call = [(s, j) for s in own for j in range(int(w.n_spans[s]))]
            assert o[r].write_embeddings(*write_args(w, call), [bits16(workloads.span_values(w, s, j)) for s, j in call], w.src_dtype) == 0
            assert o[r].set_span_grids(*_grids(w, own)) == 0
        table = bits16(workloads.embed_table(w))
        for r in (0, 1):
            assert o[r].import_mapping(o[1 - r].export_mapping()[1], o[1 - r]) == 0
            assert o[r].import_samples(_own(w, 1 - r), o[1 - r].export_samples(_own(w, 1 - r))[1]) == 0
            rc, oplan = o[r].plan_microbatches(list(range(w.n_samples)), PlanConfig(**plan_config_fields(w)))
            assert rc == 0
            oa = oplan.arrays()
            pa, rows_g, cu_g, pos_g = got[r]
            for k in ("mb_sample_off", "mb_samples", "mb_tokens", "mb_cost", "mb_bucket", "mb_rank", "rank_mb_off", "rank_mbs", "sample_mb"):
                assert np.array_equal(pa[k], oa[k]), (r, k)
                assert np.array_equal(pa[k], got[0][0][k]), k          # the same plan in both processes
            mine = [int(j) for j in oa["rank_mbs"][oa["rank_mb_off"][r]:oa["rank_mb_off"][r + 1]]]
            assert mine, "both ranks get a share in this configuration"
            rows = int(oa["mb_tokens"][mine].sum())
            n_cu = int(sum(int(oa["mb_sample_off"][j + 1] - oa["mb_sample_off"][j]) + 1 for j in mine))
            oout = np.full((rows, w.hidden), 0xFFFF, np.uint16)
            ocu = np.full(n_cu, -7, np.int32)
            opos = np.full(rows, -7, np.int32)
            assert o[r].gather_list(oplan, mine, table, oout, ocu, opos) == 0
            assert np.array_equal(rows_g, oout) and np.array_equal(cu_g, ocu) and np.array_equal(pos_g, opos), r
            oplan.destroy()
        covered = sorted(int(j) for r in (0, 1) for j in got[r][0]["rank_mbs"][got[r][0]["rank_mb_off"][r]:got[r][0]["rank_mb_off"][r + 1]])
        assert covered == list(range(len(got[0][0]["mb_tokens"])))          # the two shares are the whole plan
        for r in (0, 1):
            o[r].destroy()
    finally:
        if child.is_alive():
            child.join(timeout=30)
            if child.is_alive():
                child.kill()   # this very process object, nothing else
