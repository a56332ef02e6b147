"""GPU parity for the backbone-side outputs: the padded layout, three-component positions, ids, labels, loss
mask and the ordered table gradient, against the CPU oracle on the same seeded inputs.  Integer, copy and
order-fixed fp32 additions only, so the bar is bit-exact."""
import numpy as np
import pytest
import torch

import workloads
from harness import bits16, plan_config_fields, pool_config_fields, register_args, write_args
from oracle import OraclePool, PlanConfig, PoolConfig

pytestmark = pytest.mark.gpu


def _gpu():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    import gpu_harness
    return gpu_harness


def grid_items(w):
    items = [(s, j, workloads.span_grid(w, s, j)) for s in range(w.n_samples) for j in range(int(w.n_spans[s]))]
    items = [it for it in items if it[2] is not None]
    return [s for s, _, _ in items], [j for _, j, _ in items], [g for _, _, g in items]


class OracleSide:
    """Oracle pool fed the device's own source tensors, kept alive for range-by-range comparison."""

    def __init__(self, w, srcs):
        self.w = w
        self.pool = pool = OraclePool(PoolConfig(**pool_config_fields(w)))
        assert pool.rc == 0
        for call in w.write_calls:
            samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
            assert pool.register_samples(*register_args(w, samples)) == 0
            assert pool.write_embeddings(*write_args(w, call), [srcs[c] for c in call], w.src_dtype) == 0
        assert pool.set_span_grids(*grid_items(w)) == 0
        rc, self.plan = pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), PlanConfig(**plan_config_fields(w)))
        assert rc == 0
        self.a = self.plan.arrays()

    def padded(self, b, e, table, pad_id):
        w, a = self.w, self.a
        rows = (e - b) * w.budget_L
        n_s = int(a["mb_sample_off"][e] - a["mb_sample_off"][b])
        o = dict(out=np.full((rows, w.hidden), 0xFFFF, np.uint16), cu=np.full(n_s + 2 * (e - b), -7, np.int32),
                 pos3=np.full((3, rows), -7, np.int32), ids=np.full(rows, -7, np.int32),
                 labels=np.full(rows, -7, np.int32), mask=np.full(rows, 7, np.uint8))
        assert self.pool.gather_padded(self.plan, b, e, table, pad_id, o["out"], o["cu"], o["pos3"], o["ids"], o["labels"], o["mask"]) == 0
        return o

    def grad(self, b, e, padded, g):
        t = np.zeros((self.w.vocab, self.w.hidden), np.float32)
        t[::7] = 0.5   # accumulates onto existing content
        assert self.pool.embed_grad(self.plan, b, e, padded, g, t) == 0
        return t

    def close(self):
        self.plan.destroy()
        self.pool.destroy()


CASES = [
    ("tiny", dict()),                                                   # one span per sample, 2 microbatches
    ("image_mix_7b", dict(n_samples=14)),                               # several spans, host tier, 7168-byte rows
    ("image_mix_7b", dict(n_samples=40, hidden=56, page_bytes=4096)),   # narrow rows: one 16-byte vector chunk per 8 columns
    ("video_heavy", dict(n_samples=6)),                                 # up to 64 gridded spans per sample
    ("host_tier_stress", dict(n_samples=3)),                            # H = 8192, fp32 source
    ("image_mix_7b", dict(n_samples=24, hidden=64, page_bytes=4096, id_skew="zipf")),   # frequent ids: long runs on one table row
]


@pytest.mark.parametrize("name,kw", CASES)
def test_padded_outputs_and_table_gradient_match_oracle(name, kw):
    gh = _gpu()
    fp = gh.fp
    w = workloads.make_workload(name, **kw)
    r = gh.CudaRun(w)
    r.run_schedule()
    assert r.pool.set_span_grids(*grid_items(w), gh.cuda_stream()) == 0
    rc, plan = r.plan()
    assert rc == 0
    a = plan.arrays()
    n_mb, L, H = int(a["n_mb"]), w.budget_L, w.hidden
    ranges = [(0, n_mb)]
    if w.vocab * H * 4 <= (256 << 20):   # sub-ranges where a table copy is small
        ranges += ([(1, n_mb)] if n_mb > 1 else []) + ([(0, 1)] if n_mb > 2 else [])
    table = workloads.embed_table(w, device="cuda")
    table_bits = bits16(table)
    pad_id = -3
    orc = OracleSide(w, {c: gh.host_bits(t) for c, t in r.srcs.items()})
    for k in ("mb_sample_off", "mb_samples", "mb_tokens"):
        assert np.array_equal(a[k], orc.a[k])
    touched = 0
    for (b, e) in ranges:
        rows = (e - b) * L
        n_s = int(a["mb_sample_off"][e] - a["mb_sample_off"][b])
        out = torch.full((rows, H), -1, dtype=torch.int16, device="cuda")
        cu = torch.full((n_s + 2 * (e - b),), -7, dtype=torch.int32, device="cuda")
        pos3 = torch.full((3, rows), -7, dtype=torch.int32, device="cuda")
        ids = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
        labels = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
        mask = torch.full((rows,), 7, dtype=torch.uint8, device="cuda")
        rc = r.pool.gather_padded(plan, b, e, table.data_ptr(), table.shape[0], pad_id, out.data_ptr(), cu.data_ptr(),
                                  pos3.data_ptr(), ids.data_ptr(), labels.data_ptr(), mask.data_ptr(), gh.cuda_stream())
        assert rc == 0, fp.STATUS.get(rc)
        torch.cuda.synchronize()
        got = dict(out=out.cpu().numpy().view(np.uint16), cu=cu.cpu().numpy(), pos3=pos3.cpu().numpy(),
                   ids=ids.cpu().numpy(), labels=labels.cpu().numpy(), mask=mask.cpu().numpy())
        exp = orc.padded(b, e, table_bits, pad_id)
        for k in ("cu", "pos3", "ids", "labels", "mask", "out"):
            assert np.array_equal(got[k], exp[k]), (k, b, e)
        del out, got, exp
        for padded in (False, True):
            g_rows = rows if padded else int(a["mb_tokens"][b:e].sum())
            g = workloads.grad_values(w, 0, g_rows, device="cuda")
            gt = torch.zeros((w.vocab, H), dtype=torch.float32, device="cuda")
            gt[::7] = 0.5
            rc = r.pool.embed_grad(plan, b, e, padded, g.data_ptr(), gt.data_ptr(), w.vocab, gh.cuda_stream())
            assert rc == 0, fp.STATUS.get(rc)
            torch.cuda.synchronize()
            got_t = gt.cpu().numpy()
            exp_t = orc.grad(b, e, padded, bits16(g))
            assert np.array_equal(got_t.view(np.uint32), exp_t.view(np.uint32)), (b, e, padded)
            touched += int(np.count_nonzero(np.any(got_t[1::7] != 0, axis=1)))
            del gt, got_t, exp_t
    assert touched > 0
    assert r.pool.status() == orc.pool.status() == (0, 0)
    orc.close()
    r.close()


def test_grid_errors_and_lifetime_match_oracle():
    gh = _gpu()
    w = workloads.make_workload("tiny", n_samples=4)
    r = gh.CudaRun(w, max_samples=6)
    f = pool_config_fields(w, max_samples=6)
    op = OraclePool(PoolConfig(**f))
    r.register([0, 1])
    assert op.register_samples(*register_args(w, [0, 1])) == 0
    n0 = int(w.spans_of(0)[1][0])
    calls = [
        ([0], [0], [[1, 1, n0]]),            # fine
        ([0], [0], [[1, 2, n0]]),            # wrong product
        ([0], [0], [[0, 1, n0]]),            # zero extent
        ([0], [1], [[1, 1, n0]]),            # no such span
        ([2], [0], [[1, 1, n0]]),            # slot not registered
        ([7], [0], [[1, 1, n0]]),            # slot out of range
        ([0], [0], [[65536, 65536, 1]]),     # product wraps 32 bits: still rejected
        ([], [], np.zeros((0, 3))),          # empty call
        ([0, 1, 0], [0, 0, 0], [[1, n0, 1], [1, 1, int(w.spans_of(1)[1][0])], [n0, 1, 1]]),   # a span named twice: the last item stays
    ]
    for slots, spans, grids in calls:
        assert r.pool.set_span_grids(slots, spans, grids, gh.cuda_stream()) == op.set_span_grids(slots, spans, grids)
    # a freed and re-registered slot starts without grids
    r.write([(0, 0), (1, 0)])
    assert op.write_embeddings(*write_args(w, [(0, 0), (1, 0)]), [gh.host_bits(r.srcs[(0, 0)]), gh.host_bits(r.srcs[(1, 0)])], w.src_dtype) == 0
    assert r.pool.free([0], gh.cuda_stream()) == op.free([0]) == 0
    r.register([0])
    assert op.register_samples(*register_args(w, [0])) == 0
    r.write([(0, 0)])
    assert op.write_embeddings(*write_args(w, [(0, 0)]), [gh.host_bits(r.srcs[(0, 0)])], w.src_dtype) == 0
    cfg = plan_config_fields(w)
    rc, plan = r.pool.plan_microbatches(np.array([0, 1], np.uint32), gh.fp.PlanConfig(**cfg), gh.cuda_stream())
    rc2, oplan = op.plan_microbatches([0, 1], PlanConfig(**cfg))
    assert rc == rc2 == 0
    n_mb, L, H = plan.summary()[0], w.budget_L, w.hidden
    rows = n_mb * L
    table = workloads.embed_table(w, device="cuda")
    pos3 = torch.full((3, rows), -7, dtype=torch.int32, device="cuda")
    out = torch.empty((rows, H), dtype=torch.int16, device="cuda")
    cu = torch.empty((2 + 2 * n_mb,), dtype=torch.int32, device="cuda")
    ids, labels = (torch.empty((rows,), dtype=torch.int32, device="cuda") for _ in range(2))
    mask = torch.empty((rows,), dtype=torch.uint8, device="cuda")
    assert r.pool.gather_padded(plan, 0, n_mb, table.data_ptr(), w.vocab, 0, out.data_ptr(), cu.data_ptr(), pos3.data_ptr(),
                                ids.data_ptr(), labels.data_ptr(), mask.data_ptr(), gh.cuda_stream()) == 0
    torch.cuda.synchronize()
    o = dict(out=np.zeros((rows, H), np.uint16), cu=np.zeros(2 + 2 * n_mb, np.int32), pos3=np.zeros((3, rows), np.int32),
             ids=np.zeros(rows, np.int32), labels=np.zeros(rows, np.int32), mask=np.zeros(rows, np.uint8))
    assert op.gather_padded(oplan, 0, n_mb, bits16(table), 0, o["out"], o["cu"], o["pos3"], o["ids"], o["labels"], o["mask"]) == 0
    assert np.array_equal(pos3.cpu().numpy(), o["pos3"])
    # argument errors of the two consumer calls
    assert r.pool.gather_padded(plan, 1, 0, table.data_ptr(), w.vocab, 0, out.data_ptr(), cu.data_ptr(), pos3.data_ptr(),
                                ids.data_ptr(), labels.data_ptr(), mask.data_ptr(), gh.cuda_stream()) == -1
    assert r.pool.gather_padded(plan, 0, n_mb, table.data_ptr(), w.vocab, 0, out.data_ptr(), cu.data_ptr(), 0,
                                ids.data_ptr(), labels.data_ptr(), mask.data_ptr(), gh.cuda_stream()) == -1
    assert r.pool.embed_grad(plan, 0, n_mb + 1, False, out.data_ptr(), out.data_ptr(), w.vocab, gh.cuda_stream()) == -1
    assert r.pool.embed_grad(plan, 0, n_mb, False, 0, out.data_ptr(), w.vocab, gh.cuda_stream()) == -1
    assert r.pool.embed_grad(plan, 0, 0, False, 0, 0, w.vocab, gh.cuda_stream()) == 0
    assert r.pool.free([1], gh.cuda_stream()) == 0
    assert r.pool.embed_grad(plan, 0, n_mb, False, out.data_ptr(), out.data_ptr(), w.vocab, gh.cuda_stream()) == -5   # plan died with its sample
    assert r.pool.status() == (0, 0)
    oplan.destroy(); op.destroy()
    r.close()


def test_bad_token_id_in_gradient_is_reported_and_skipped():
    gh = _gpu()
    w = workloads.make_workload("tiny", n_samples=3)
    r = gh.CudaRun(w)
    r.run_schedule()
    rc, plan = r.plan()
    a = plan.arrays()
    n_mb, H = int(a["n_mb"]), w.hidden
    rows = int(a["mb_tokens"].sum())
    small_vocab = 1000   # most ids are outside
    g = workloads.grad_values(w, 0, rows, device="cuda")
    gt = torch.zeros((small_vocab, H), dtype=torch.float32, device="cuda")
    assert r.pool.embed_grad(plan, 0, n_mb, False, g.data_ptr(), gt.data_ptr(), small_vocab, gh.cuda_stream()) == 0
    torch.cuda.synchronize()
    code, detail = r.pool.status()
    exp_pool = OraclePool(PoolConfig(**pool_config_fields(w)))
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        exp_pool.register_samples(*register_args(w, samples))
        exp_pool.write_embeddings(*write_args(w, call), [gh.host_bits(r.srcs[c]) for c in call], w.src_dtype)
    rc, oplan = exp_pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), PlanConfig(**plan_config_fields(w)))
    et = np.zeros((small_vocab, H), np.float32)
    assert exp_pool.embed_grad(oplan, 0, n_mb, False, bits16(g), et) == 0
    assert (code, detail) == exp_pool.status() and code == -9
    assert np.array_equal(gt.cpu().numpy().view(np.uint32), et.view(np.uint32))
    oplan.destroy(); exp_pool.destroy()
    r.close()
