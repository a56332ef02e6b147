"""Two processes' segments of one GVA space, emulated as two pools in one process on one GPU (no kernel of one
pool ever waits on the other): the producer writes, exports its mapping and its samples' descriptors; the
consumer imports both and assembles microbatches that mix its own samples with the producer's, reading the
producer's pages in place.  Every status code and every assembled byte must equal the oracle's."""
import numpy as np
import pytest
import torch

import workloads
from harness import bits16, plan_config_fields, pool_config_fields, register_args, write_args
from oracle import OraclePool, PlanConfig, PoolConfig

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("peers_remote", [0, 1])
@pytest.mark.parametrize("name,kw", [
    ("image_mix_7b", dict(n_samples=10, hidden=56, page_bytes=4096)),
    ("image_mix_7b", dict(n_samples=12, hidden=3584)),                    # 2 MiB pages, both tiers on both sides
    ("host_tier_stress", dict(n_samples=4, hidden=1024, page_bytes=65536)),
])
def test_consumer_reads_producer_pages_in_place(name, kw, peers_remote):
    """peers_remote = 1: the consumer treats the producer's HBM frames as another GPU's (they get the separate
    bulk-copy launch that frames behind NVLink get), which must not change a byte."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import cuda_stream
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload(name, **kw)
    w.budget_L = max(w.budget_L // 4, w.max_seq_len)
    n = w.n_samples
    remote = list(range(0, n, 2))
    local = list(range(1, n, 2))[:-1]

    def cfg(rank):
        f = pool_config_fields(w, max_samples=2 * n)
        f.update(world_size=2, rank=rank, bind_seed=100 + rank, ring_seed=200 + rank, max_imported_pages=w.hbm_pages + w.host_pages)
        return f
    g = {r: fp.Pool(fp.PoolConfig(**cfg(r))) for r in (0, 1)}
    o = {r: OraclePool(PoolConfig(**cfg(r))) for r in (0, 1)}
    assert all(p.rc == 0 for p in g.values()) and all(p.rc == 0 for p in o.values())
    # (with peers_remote = 1 both pools also send their own host tier through the copy engines; a plan that holds an
    # imported sample still assembles with the kernels)
    assert g[0].set_tuning(peers_remote=peers_remote, remote_ctas=3, host_copy_engine=peers_remote) == 0 and g[0].get_tuning()["peers_remote"] == peers_remote
    assert g[1].set_tuning(host_copy_engine=peers_remote) == 0
    g[0].profile_enable(True)
    keep = []

    def fill(rank, samples):
        a = register_args(w, samples)
        ids = torch.from_numpy(a[5]).cuda(); keep.append(ids)
        assert g[rank].register_samples(*a[:5], ids.data_ptr(), cuda_stream()) == o[rank].register_samples(*a) == 0
        call = [(s, j) for s in samples for j in range(int(w.n_spans[s]))]
        srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]; keep.append(srcs)
        assert g[rank].write_embeddings(*write_args(w, call), [t.data_ptr() for t in srcs], w.src_dtype, cuda_stream()) == 0
        host = [bits16(t) if w.src_dtype == 0 else t.view(torch.int32).cpu().numpy().view(np.uint32) for t in srcs]
        assert o[rank].write_embeddings(*write_args(w, call), host, w.src_dtype) == 0
        gi = [(s, j, workloads.span_grid(w, s, j)) for s, j in call]
        gi = [t for t in gi if t[2] is not None]
        ga_ = ([s for s, _, _ in gi], [j for _, j, _ in gi], [t for _, _, t in gi])
        assert g[rank].set_span_grids(*ga_, cuda_stream()) == o[rank].set_span_grids(*ga_) == 0

    fill(1, remote)
    fill(0, local)
    # before the mapping is known the producer's GVAs do not translate on the consumer
    gva = [o[1].page_gva(0), o[0].page_gva(0)]
    assert list(g[0].translate(gva)[0]) == [-7, 0]
    rc_g, sblob_g = g[1].export_samples(remote, cuda_stream())
    rc_o, sblob_o = o[1].export_samples(remote)
    assert rc_g == rc_o == 0
    loc = list(range(n, n + len(remote)))
    assert g[0].import_samples(loc, sblob_g, cuda_stream()) == o[0].import_samples(loc, sblob_o) == -1
    rc, mblob = g[1].export_mapping()
    assert rc == 0
    hbm, host, text = g[1].backing()
    assert g[0].import_mapping(mblob[:-4], hbm, host, text) == -1
    assert g[0].import_mapping(mblob, hbm, host, text) == 0
    assert g[0].import_mapping(mblob, hbm, host, text) == -10
    assert o[0].import_mapping(o[1].export_mapping()[1], o[1]) == 0
    # translation of the producer's pages on the consumer = the oracle's
    P = w.hbm_pages + w.host_pages
    gvas = [o[1].page_gva(k) + 32 for k in range(0, P, max(1, P // 64))]
    st, kind, frame, off = g[0].translate(gvas)
    for i, gv in enumerate(gvas):
        rc, proc, k, fr, of = o[0].translate_ex(gv)
        assert (int(st[i]), int(kind[i]), int(frame[i]), int(off[i])) == (rc, k, fr, of) and proc == 1
    assert g[1].export_samples([remote[0], 2 * n - 1], cuda_stream())[0] == o[1].export_samples([remote[0], 2 * n - 1])[0] == -3
    bad = [loc[0], local[0]] + loc[2:]
    assert g[0].import_samples(bad, sblob_g, cuda_stream()) == o[0].import_samples(bad, sblob_o) == -10
    assert g[0].import_samples(loc, sblob_g, cuda_stream()) == o[0].import_samples(loc, sblob_o) == 0
    for l, r in zip(loc, remote):
        for j in range(int(w.n_spans[r])):
            assert np.array_equal(g[0].span_pages(l, j)[1], o[1].span_pages(r, j)[1])
    ring_before = g[0].ring().copy()
    # microbatches that mix own and imported samples
    order = [x for pair in zip(loc, local + loc[len(local):]) for x in pair]
    order = list(dict.fromkeys(order + loc + local))
    pc = plan_config_fields(w)
    rc1, gp = g[0].plan_microbatches(order, fp.PlanConfig(**pc), cuda_stream())
    rc2, op = o[0].plan_microbatches(order, PlanConfig(**pc))
    assert rc1 == rc2 == 0
    ga, oa = gp.arrays(), op.arrays()
    for k in ("mb_sample_off", "mb_samples", "mb_tokens", "mb_cost", "mb_bucket", "mb_rank", "rank_mbs", "sample_mb"):
        assert np.array_equal(ga[k], oa[k]), k
    n_mb, total, _ = gp.summary()
    table = workloads.embed_table(w, device="cuda")
    out = torch.full((total, w.hidden), -1, dtype=torch.int16, device="cuda")
    cu = torch.full((len(order) + n_mb,), -1, dtype=torch.int32, device="cuda")
    pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
    assert g[0].gather_packed(gp, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), cuda_stream()) == 0
    oout = np.full((total, w.hidden), 0xFFFF, np.uint16); ocu = np.full(len(order) + n_mb, -1, np.int32); opos = np.full(total, -1, np.int32)
    assert o[0].gather_packed(op, 0, n_mb, bits16(table), oout, ocu, opos) == 0
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint16)
    assert np.array_equal(got, oout) and not np.any(np.all(got == 0xFFFF, axis=1))
    assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos)
    assert g[0].status() == o[0].status() == (0, 0)
    prof = g[0].profile_read()
    assert (prof["gather_remote"]["launches"] > 0) == bool(peers_remote) and prof["gather_device"]["launches"] > 0
    # backbone-side outputs over the same mixed microbatches: the imported spans' token grids came with the descriptors
    L = w.budget_L
    rows = n_mb * L
    p_out = torch.full((rows, w.hidden), -1, dtype=torch.int16, device="cuda")
    p_cu = torch.full((len(order) + 2 * n_mb,), -7, dtype=torch.int32, device="cuda")
    p_pos3 = torch.full((3, rows), -7, dtype=torch.int32, device="cuda")
    p_ids, p_lab = (torch.full((rows,), -7, dtype=torch.int32, device="cuda") for _ in range(2))
    p_msk = torch.full((rows,), 7, dtype=torch.uint8, device="cuda")
    assert g[0].gather_padded(gp, 0, n_mb, table.data_ptr(), w.vocab, -1, p_out.data_ptr(), p_cu.data_ptr(), p_pos3.data_ptr(),
                              p_ids.data_ptr(), p_lab.data_ptr(), p_msk.data_ptr(), cuda_stream()) == 0
    e = dict(out=np.full((rows, w.hidden), 0xFFFF, np.uint16), cu=np.full(len(order) + 2 * n_mb, -7, np.int32),
             pos3=np.full((3, rows), -7, np.int32), ids=np.full(rows, -7, np.int32), labels=np.full(rows, -7, np.int32),
             mask=np.full(rows, 7, np.uint8))
    assert o[0].gather_padded(op, 0, n_mb, bits16(table), -1, e["out"], e["cu"], e["pos3"], e["ids"], e["labels"], e["mask"]) == 0
    torch.cuda.synchronize()
    for key, t in (("out", p_out), ("cu", p_cu), ("pos3", p_pos3), ("ids", p_ids), ("labels", p_lab), ("mask", p_msk)):
        got_k = t.cpu().numpy()
        assert np.array_equal(got_k.view(np.uint16) if key == "out" else got_k, e[key]), key
    # an imported gridded span shows in the positions (the three components differ somewhere inside an imported sample)
    row = 0
    imported_rows = []
    for j in range(n_mb):
        row = j * L
        for slot in oa["mb_samples"][oa["mb_sample_off"][j]:oa["mb_sample_off"][j + 1]]:
            ln = int(w.seq_len[remote[loc.index(int(slot))]]) if int(slot) in loc else int(w.seq_len[int(slot)])
            if int(slot) in loc:
                imported_rows.append((row, row + ln))
            row += ln
    assert any(np.any(e["pos3"][0, a:b] != e["pos3"][2, a:b]) for a, b in imported_rows)
    grad = workloads.grad_values(w, 0, total, device="cuda")
    gt = torch.zeros((w.vocab, w.hidden), dtype=torch.float32, device="cuda")
    assert g[0].embed_grad(gp, 0, n_mb, False, grad.data_ptr(), gt.data_ptr(), w.vocab, cuda_stream()) == 0
    et = np.zeros((w.vocab, w.hidden), np.float32)
    assert o[0].embed_grad(op, 0, n_mb, False, bits16(grad), et) == 0
    torch.cuda.synchronize()
    assert np.array_equal(gt.cpu().numpy().view(np.uint32), et.view(np.uint32))
    assert g[0].status() == o[0].status() == (0, 0)
    # freeing imports returns nothing to the consumer's rings, and the plan dies with them
    assert g[0].free(loc, cuda_stream()) == o[0].free(loc) == 0
    assert np.array_equal(g[0].ring(), ring_before) and np.array_equal(g[0].ring(), o[0].ring())
    assert g[0].stats()["pages_free"] == o[0].free_pages()[0]
    assert g[0].gather_packed(gp, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), cuda_stream()) == -5
    assert g[0].free(local, cuda_stream()) == o[0].free(local) == 0
    assert g[1].free(remote, cuda_stream()) == o[1].free(remote) == 0
    for r in (0, 1):
        assert np.array_equal(g[r].ring(), o[r].ring())
        assert g[r].stats()["pages_free"] == P and g[r].stats()["text_pages_free"] == o[r].free_pages()[1]
    for r in (0, 1):
        g[r].destroy(); o[r].destroy()
