"""The decoupled producer-consumer flow on two streams: the producer stream registers and writes batch k+1 while
the consumer stream plans and assembles batch k; pages and slots are recycled (pool_free on the producer stream)
as soon as their microbatches are assembled.  The library orders the two streams itself.  Ready-queue answers,
status codes, page assignment and every assembled byte must equal the oracle's sequential execution of the same
calls."""
import numpy as np
import pytest
import torch

import workloads
from harness import bits16, plan_config_fields, pool_config_fields, register_args, write_args
from oracle import OraclePool, PlanConfig, PoolConfig

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("copy_engine", [0, 1])   # 1: the host tier through the copy engines, both directions at once
@pytest.mark.parametrize("name,kw,group", [
    ("image_mix_7b", dict(n_samples=48, hidden=512, page_bytes=65536), 8),
    ("host_tier_stress", dict(n_samples=12, hidden=1024, page_bytes=65536), 3),
])
def test_overlapped_write_and_gather_match_sequential_oracle(name, kw, group, copy_engine):
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload(name, **kw)
    f = pool_config_fields(w, max_samples=2 * group)          # slots are recycled
    need = sorted((sum(w.pages_of_span(t) for t in w.spans_of(s)[1]) for s in range(w.n_samples)), reverse=True)
    cap = sum(need[:2 * group]) + 2                            # room for two groups in flight, no more
    f["hbm_pages"], f["host_pages"] = (cap + 1) // 2, cap // 2
    pool, opool = fp.Pool(fp.PoolConfig(**f)), OraclePool(PoolConfig(**f))
    assert pool.rc == 0 and opool.rc == 0
    assert pool.set_tuning(host_copy_engine=copy_engine) == 0
    prod, cons = torch.cuda.Stream(), torch.cuda.Stream()
    table = workloads.embed_table(w, device="cuda")
    table_h = bits16(table)
    pc = plan_config_fields(w)
    keep, results = [], []
    groups = [list(range(g, min(g + group, w.n_samples))) for g in range(0, w.n_samples, group)]

    def slot_of(s):
        return s % (2 * group)

    def produce(samples):
        a = list(register_args(w, samples))
        a[0] = np.array([slot_of(s) for s in samples], dtype=np.uint32)
        call = [(s, j) for s in samples for j in range(int(w.n_spans[s]))]
        slots = np.array([slot_of(s) for s, _ in call], dtype=np.uint32)
        _, span_idx, ntok = write_args(w, call)
        with torch.cuda.stream(prod):
            ids = torch.from_numpy(a[5]).cuda(); keep.append(ids)
            srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]; keep.append(srcs)
            g1 = pool.register_samples(*a[:5], ids.data_ptr(), prod.cuda_stream)
            g2 = pool.write_embeddings(slots, span_idx, ntok, [t.data_ptr() for t in srcs], w.src_dtype, prod.cuda_stream)
        host = [bits16(t) if w.src_dtype == 0 else t.view(torch.int32).cpu().numpy().view(np.uint32) for t in srcs]
        assert (g1, g2) == (opool.register_samples(*a), opool.write_embeddings(slots, span_idx, ntok, host, w.src_dtype)) == (0, 0)

    def consume():
        rc_g, slots_g, tok_g = pool.take_ready(1, group)     # one batch per round, in completion order
        rc_o, slots_o, tok_o = opool.take_ready(1, group)
        assert rc_g == rc_o == 0 and list(slots_g) == list(slots_o) and tok_g == tok_o
        with torch.cuda.stream(cons):
            rc1, gp = pool.plan_microbatches(slots_g, fp.PlanConfig(**pc), cons.cuda_stream)
            n_mb, total, _ = gp.summary()
            out = torch.full((total, w.hidden), -1, dtype=torch.int16, device="cuda")
            cu = torch.full((len(slots_g) + n_mb,), -1, dtype=torch.int32, device="cuda")
            pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
            rc2 = pool.gather_packed(gp, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), cons.cuda_stream)
        rc3, op = opool.plan_microbatches(slots_o, PlanConfig(**pc))
        oout = np.full((total, w.hidden), 0xFFFF, np.uint16); ocu = np.full(len(slots_o) + n_mb, -1, np.int32); opos = np.full(total, -1, np.int32)
        rc4 = opool.gather_packed(op, 0, n_mb, table_h, oout, ocu, opos)
        assert (rc1, rc2, rc3, rc4) == (0, 0, 0, 0)
        # recycle at once, on the producer stream: the library makes the free wait for the gather
        assert pool.free(slots_g, prod.cuda_stream) == opool.free(slots_o) == 0
        results.append((out, cu, pos, oout, ocu, opos, gp))

    produce(groups[0])
    for k in range(len(groups)):
        if k + 1 < len(groups):
            produce(groups[k + 1])        # enqueued before batch k is assembled: they overlap on the device
        consume()
    torch.cuda.synchronize()
    for out, cu, pos, oout, ocu, opos, gp in results:
        got = out.cpu().numpy().view(np.uint16)
        assert np.array_equal(got, oout) and not np.any(np.all(got == 0xFFFF, axis=1))
        assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos)
        gp.destroy()
    assert pool.status() == opool.status() == (0, 0)
    assert np.array_equal(pool.ring(), opool.ring())
    assert pool.ready_count() == opool.ready_count()
    pool.destroy(); opool.destroy()
