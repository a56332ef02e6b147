"""Pins for the oracle's multi-process GVA space (Sec. 3.2: per-process segments, exported mappings, local
translation) -- CPU only.  The new code is reduced to what is already pinned: a consumer that imports a
producer's mapping and samples must assemble exactly what the producer assembles itself."""
import numpy as np

import workloads
from harness import bits16, host_span, plan_config_fields, pool_config_fields, register_args, write_args
from oracle import OraclePool, PlanConfig, PoolConfig


def make_rank(w, rank, world=3, **over):
    f = pool_config_fields(w, max_samples=w.n_samples * 2)
    f.update(world_size=world, rank=rank, bind_seed=100 + rank, ring_seed=200 + rank)
    f.update(over)
    p = OraclePool(PoolConfig(**f))
    assert p.rc == 0
    return p


def fill(pool, w, samples):
    assert pool.register_samples(*register_args(w, samples)) == 0
    call = [(s, j) for s in samples for j in range(int(w.n_spans[s]))]
    assert pool.write_embeddings(*write_args(w, call), [host_span(w, s, j) for s, j in call], w.src_dtype) == 0
    grids = [(s, j, workloads.span_grid(w, s, j)) for s, j in call]
    grids = [t for t in grids if t[2] is not None]
    assert pool.set_span_grids([s for s, _, _ in grids], [j for _, j, _ in grids], [g for _, _, g in grids]) == 0


def padded_all(pool, plan, w, table, n_slots):
    n_mb = plan.summary()[0]
    rows = n_mb * w.budget_L
    o = dict(out=np.full((rows, w.hidden), 0xFFFF, np.uint16), cu=np.full(n_slots + 2 * n_mb, -7, np.int32),
             pos3=np.full((3, rows), -7, np.int32), ids=np.full(rows, -7, np.int32), labels=np.full(rows, -7, np.int32),
             mask=np.full(rows, 7, np.uint8))
    assert pool.gather_padded(plan, 0, n_mb, table, -1, o["out"], o["cu"], o["pos3"], o["ids"], o["labels"], o["mask"]) == 0
    return o


def gather_all(pool, slots, w, table):
    rc, plan = pool.plan_microbatches(slots, PlanConfig(**plan_config_fields(w)))
    assert rc == 0
    n_mb, total, _ = plan.summary()
    out = np.full((total, w.hidden), 0xFFFF, np.uint16)
    cu = np.full(len(slots) + n_mb, -1, np.int32)
    pos = np.full(total, -1, np.int32)
    rc = pool.gather_packed(plan, 0, n_mb, table, out, cu, pos)
    return rc, out, cu, pos, plan


def test_segments_are_disjoint_and_follow_the_formula():
    w = workloads.make_workload("image_mix_7b", n_samples=4, hidden=64, page_bytes=4096)
    pools = [make_rank(w, r) for r in range(3)]
    M, PS = 1 << 40, 4096
    for r, p in enumerate(pools):
        assert p.page_gva(0) == (1 << 44) + r * M and p.page_gva(3) == (1 << 44) + r * M + 3 * PS
        assert p.page_gva(w.hbm_pages) == (1 << 45) + r * M          # first DRAM page of process r
        # before any import, only the own segment translates
        for q in range(3):
            rc = p.translate_ex(pools[q].page_gva(0))[0]
            assert rc == (0 if q == r else -7)
    for p in pools:
        p.destroy()


def test_imported_mapping_translates_like_the_owner():
    w = workloads.make_workload("image_mix_7b", n_samples=4, hidden=64, page_bytes=4096)
    a, b = make_rank(w, 0, world=2), make_rank(w, 1, world=2)
    rc, blob = b.export_mapping()
    assert rc == 0
    assert a.import_mapping(blob[:-8], b) == -1                      # truncated blob
    assert a.import_mapping(a.export_mapping()[1], a) == -1          # own rank
    other = make_rank(w, 1, world=2, max_size=1 << 39)
    assert a.import_mapping(other.export_mapping()[1], other) == -1  # another GVA space
    assert a.import_mapping(blob, None) == -1                        # no way to reach the peer's frames
    assert a.import_mapping(blob, b) == 0
    assert a.import_mapping(blob, b) == -10                          # that process is known already
    P = w.hbm_pages + w.host_pages
    for g in range(P):
        gva = b.page_gva(g)
        rc, proc, kind, frame, off = a.translate_ex(gva + 40)
        assert (rc, proc, off) == (0, 1, 40)
        assert (kind, frame) == b.translate(gva)[1:3]                # the owner's own answer
    assert a.translate_ex(b.page_gva(0) + (P + 4) * 4096 * 1000)[0] == -7
    for p in (a, b, other):
        p.destroy()


def test_consumer_assembles_what_the_producer_would():
    w = workloads.make_workload("image_mix_7b", n_samples=10, hidden=56, page_bytes=4096)
    w.budget_L = 12000
    table = bits16(workloads.embed_table(w))
    prod, cons = make_rank(w, 1, world=2), make_rank(w, 0, world=2)
    remote, local = [0, 2, 4, 6, 8], [1, 3, 5]
    fill(prod, w, remote)
    fill(cons, w, local)
    cons_ring, prod_ring = cons.ring().copy(), prod.ring().copy()
    assert cons.import_samples([10, 11], prod.export_samples([0, 2])[1]) == -1       # mapping not imported yet
    assert cons.import_mapping(prod.export_mapping()[1], prod) == 0
    assert prod.export_samples([0, 9])[0] == -3 and prod.export_samples([0, 0])[0] == -1
    rc, blob = prod.export_samples(remote)
    assert rc == 0
    assert cons.import_samples([10, 1, 12, 13, 14], blob) == -10                     # slot 1 is taken
    assert cons.import_samples([10, 11, 12, 13], blob) == -1                         # count mismatch
    assert cons.import_samples([10, 11, 12, 13, 14], blob) == 0
    assert cons.write_embeddings([10], [0], [int(w.spans_of(0)[1][0])], [host_span(w, 0, 0)], 0) == -4
    # the same mix of samples, assembled by a single process that holds everything (already pinned path) ...
    ref = make_rank(w, 0, world=1)
    fill(ref, w, remote)
    fill(ref, w, local)
    order_ref = [0, 1, 2, 3, 4, 5, 6, 8]
    rc, out_ref, cu_ref, pos_ref, plan_ref = gather_all(ref, order_ref, w, table)
    assert rc == 0
    # ... equals what the consumer assembles from its own samples plus the imported ones
    order_cons = [10, 1, 11, 3, 12, 5, 13, 14]                                       # same samples, same order
    rc, out, cu, pos, plan = gather_all(cons, order_cons, w, table)
    assert rc == 0 and cons.status() == (0, 0)
    assert np.array_equal(out, out_ref) and np.array_equal(cu, cu_ref) and np.array_equal(pos, pos_ref)
    a, b = plan.arrays(), plan_ref.arrays()
    for k in ("mb_sample_off", "mb_tokens", "mb_cost", "mb_rank", "sample_mb"):
        assert np.array_equal(a[k], b[k])
    # the spans' token grids travel with the descriptors: positions, labels and the table gradient are the single process's
    po, pr = padded_all(cons, plan, w, table, len(order_cons)), padded_all(ref, plan_ref, w, table, len(order_ref))
    for k in po:
        assert np.array_equal(po[k], pr[k]), k
    assert np.any(po["pos3"][0] != po["pos3"][2])
    grad = bits16(workloads.grad_values(w, 0, out.shape[0]))
    t_c, t_r = np.zeros((w.vocab, w.hidden), np.float32), np.zeros((w.vocab, w.hidden), np.float32)
    assert cons.embed_grad(plan, 0, plan.summary()[0], False, grad, t_c) == 0
    assert ref.embed_grad(plan_ref, 0, plan_ref.summary()[0], False, grad, t_r) == 0
    assert np.array_equal(t_c.view(np.uint32), t_r.view(np.uint32)) and np.any(t_c != 0)
    # imported page lists are the producer's
    for loc, rem in zip([10, 11, 12, 13, 14], remote):
        for j in range(int(w.n_spans[rem])):
            assert np.array_equal(cons.span_pages(loc, j)[1], prod.span_pages(rem, j)[1])
    # freeing imports returns nothing to either process's rings; the plan dies with its samples
    assert cons.free([10, 11, 12, 13, 14]) == 0
    assert np.array_equal(cons.ring(), cons_ring) and np.array_equal(prod.ring(), prod_ring)
    assert gather_all.__call__ and cons.gather_packed(plan, 0, 1, table, out, cu, pos) == -5
    assert cons.free([1, 3, 5]) == 0 and prod.free(remote) == 0
    assert cons.free_pages()[0] == cons.cfg.hbm_pages + cons.cfg.host_pages
    for p in (prod, cons, ref):
        p.destroy()
