"""Two real processes on one node (Sec. 3.2: every process addresses every other process's segment): a producer
process writes into its own pool and hands the consumer, over a host channel, its mapping blob, its samples'
descriptors and shareable handles of its slabs; the consumer (this process) maps the slabs, imports both blobs and
assembles microbatches that mix its own samples with the producer's, reading the producer's pages in place.
Neither process's kernels ever wait on the other's.  The assembled bytes must equal the oracle's two-pool run."""
import multiprocessing as mp
import queue

import numpy as np
import pytest
import torch

import workloads
from harness import bits16, plan_config_fields, pool_config_fields, register_args, write_args

pytestmark = pytest.mark.gpu

KW = dict(n_samples=12, hidden=512, page_bytes=65536, all_hbm=True)


def _cfg(w, rank):
    f = pool_config_fields(w, max_samples=2 * w.n_samples)
    f.update(world_size=2, rank=rank, bind_seed=100 + rank, ring_seed=200 + rank, max_imported_pages=w.hbm_pages + w.host_pages)
    return f


def _fill(pool, w, samples, stream, keep):
    """register + write + grids of `samples` on a CUDA pool; returns host copies of the sources."""
    a = register_args(w, samples)
    ids = torch.from_numpy(a[5]).cuda()
    keep.append(ids)
    assert pool.register_samples(*a[:5], ids.data_ptr(), stream) == 0
    call = [(s, j) for s in samples for j in range(int(w.n_spans[s]))]
    srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]
    keep.append(srcs)
    assert pool.write_embeddings(*write_args(w, call), [t.data_ptr() for t in srcs], w.src_dtype, stream) == 0
    gi = [(s, j, workloads.span_grid(w, s, j)) for s, j in call]
    gi = [t for t in gi if t[2] is not None]
    assert pool.set_span_grids([s for s, _, _ in gi], [j for _, j, _ in gi], [g for _, _, g in gi], stream) == 0
    return call, [bits16(t) for t in srcs]


def producer_main(to_consumer, from_consumer):
    """The producer process: rank 1 of the GVA space."""
    try:
        torch.cuda.set_device(0)
        from paper_2606_23087_b200 import binding as fp
        w = workloads.make_workload("image_mix_7b", **KW)
        remote = list(range(0, w.n_samples, 2))
        pool = fp.Pool(fp.PoolConfig(**_cfg(w, 1)))
        assert pool.rc == 0
        st = torch.cuda.current_stream().cuda_stream
        keep = []
        _fill(pool, w, remote, st, keep)
        torch.cuda.synchronize()
        rc1, mblob = pool.export_mapping()
        rc2, sblob = pool.export_samples(remote, st)
        rc3, handles = pool.ipc_export()
        assert rc1 == rc2 == rc3 == 0
        to_consumer.put(("ok", mblob.tobytes(), sblob.tobytes(), handles))
        from_consumer.get(timeout=300)   # the consumer has freed its imports and unmapped the slabs
        assert pool.free(remote, st) == 0
        torch.cuda.synchronize()
        assert pool.status() == (0, 0)
        pool.destroy()
        to_consumer.put(("done",))
    except BaseException as e:   # report instead of leaving the consumer waiting
        to_consumer.put(("error", repr(e)))
        raise


def test_consumer_process_reads_a_producer_process_in_place():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import cuda_stream
    from oracle import OraclePool, PlanConfig, PoolConfig
    from paper_2606_23087_b200 import binding as fp
    ctx = mp.get_context("spawn")
    to_consumer, from_consumer = ctx.Queue(), ctx.Queue()
    child = ctx.Process(target=producer_main, args=(to_consumer, from_consumer), daemon=True)
    child.start()
    try:
        w = workloads.make_workload("image_mix_7b", **KW)
        n = w.n_samples
        remote = list(range(0, n, 2))
        local = list(range(1, n, 2))
        loc = list(range(n, n + len(remote)))
        st = cuda_stream()
        cons = fp.Pool(fp.PoolConfig(**_cfg(w, 0)))
        assert cons.rc == 0
        keep = []
        call_l, host_l = _fill(cons, w, local, st, keep)
        try:
            msg = to_consumer.get(timeout=300)
        except queue.Empty:
            pytest.fail("the producer process did not answer")
        assert msg[0] == "ok", msg
        mblob, sblob, handles = (np.frombuffer(msg[1], np.uint8), np.frombuffer(msg[2], np.uint8), msg[3])
        rc, hbm, text = fp.ipc_open(handles)
        assert rc == 0 and hbm and text
        assert cons.import_mapping(mblob, hbm, 0, text) == 0
        assert cons.import_samples(loc, sblob, st) == 0
        order = [x for pair in zip(loc, local) for x in pair]
        pc = plan_config_fields(w)
        pc["budget_L"] = int(w.seq_len.max()) * 2
        rc, plan = cons.plan_microbatches(order, fp.PlanConfig(**pc), st)
        assert rc == 0
        n_mb, total, _ = plan.summary()
        table = workloads.embed_table(w, device="cuda")
        out = torch.full((total, w.hidden), -1, dtype=torch.int16, device="cuda")
        cu = torch.full((len(order) + n_mb,), -1, dtype=torch.int32, device="cuda")
        pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
        assert cons.gather_packed(plan, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), st) == 0
        rows = n_mb * pc["budget_L"]
        pos3 = torch.full((3, rows), -7, dtype=torch.int32, device="cuda")
        p_out = torch.empty((rows, w.hidden), dtype=torch.int16, device="cuda")
        p_cu = torch.empty((len(order) + 2 * n_mb,), dtype=torch.int32, device="cuda")
        p_ids, p_lab = (torch.empty((rows,), dtype=torch.int32, device="cuda") for _ in range(2))
        p_msk = torch.empty((rows,), dtype=torch.uint8, device="cuda")
        assert cons.gather_padded(plan, 0, n_mb, table.data_ptr(), w.vocab, -1, p_out.data_ptr(), p_cu.data_ptr(), pos3.data_ptr(),
                                  p_ids.data_ptr(), p_lab.data_ptr(), p_msk.data_ptr(), st) == 0
        torch.cuda.synchronize()
        assert cons.status() == (0, 0)
        # the oracle's two pools, in this process (the generator gives the producer's sources again)
        o = {r: OraclePool(PoolConfig(**_cfg(w, r))) for r in (0, 1)}
        for rank, samples in ((1, remote), (0, local)):
            assert o[rank].register_samples(*register_args(w, samples)) == 0
            call = [(s, j) for s in samples for j in range(int(w.n_spans[s]))]
            assert o[rank].write_embeddings(*write_args(w, call), [bits16(workloads.span_values(w, s, j)) for s, j in call], w.src_dtype) == 0
            gi = [(s, j, workloads.span_grid(w, s, j)) for s, j in call]
            gi = [t for t in gi if t[2] is not None]
            assert o[rank].set_span_grids([s for s, _, _ in gi], [j for _, j, _ in gi], [g for _, _, g in gi]) == 0
        assert o[0].import_mapping(o[1].export_mapping()[1], o[1]) == 0
        assert o[0].import_samples(loc, o[1].export_samples(remote)[1]) == 0
        rc, oplan = o[0].plan_microbatches(order, PlanConfig(**pc))
        assert rc == 0 and oplan.summary() == plan.summary()
        oout = np.full((total, w.hidden), 0xFFFF, np.uint16)
        ocu = np.full(len(order) + n_mb, -1, np.int32)
        opos = np.full(total, -1, np.int32)
        assert o[0].gather_packed(oplan, 0, n_mb, bits16(table), oout, ocu, opos) == 0
        assert np.array_equal(out.cpu().numpy().view(np.uint16), oout)
        assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos)
        e = dict(out=np.zeros((rows, w.hidden), np.uint16), cu=np.zeros(len(order) + 2 * n_mb, np.int32), pos3=np.zeros((3, rows), np.int32),
                 ids=np.zeros(rows, np.int32), labels=np.zeros(rows, np.int32), mask=np.zeros(rows, np.uint8))
        assert o[0].gather_padded(oplan, 0, n_mb, bits16(table), -1, e["out"], e["cu"], e["pos3"], e["ids"], e["labels"], e["mask"]) == 0
        assert np.array_equal(pos3.cpu().numpy(), e["pos3"]) and np.array_equal(p_lab.cpu().numpy(), e["labels"])
        assert np.array_equal(p_out.cpu().numpy().view(np.uint16), e["out"])
        # release in the right order: imports first, then the mapping of the producer's slabs, then the producer
        assert cons.free(loc, st) == 0 and cons.free(local, st) == 0
        torch.cuda.synchronize()
        plan.destroy(); oplan.destroy()
        cons.destroy()
        assert fp.ipc_close(hbm, text) == 0
        for r in (0, 1):
            o[r].destroy()
        from_consumer.put("go on")
        msg = to_consumer.get(timeout=120)
        assert msg[0] == "done", msg
        child.join(timeout=60)
        assert child.exitcode == 0
    finally:
        if child.is_alive():
            from_consumer.put("abort")
            child.join(timeout=30)
            if child.is_alive():
                child.kill()   # this very process object, nothing else
