"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle, element by element, on the
same seeded inputs.  Everything here is integer, index and copy work (including the fixed RNE cast), so the
bar is bit-exact: np.array_equal on every output array and equal status codes."""
import numpy as np
import pytest
import torch

import workloads
from harness import (bits16, plan_config_fields, pool_config_fields, register_args, run_oracle, write_args)
from oracle import OraclePool, PlanConfig, PoolConfig, f32_to_bf16_rne, plan_from_lengths

pytestmark = pytest.mark.gpu

PLAN_KEYS = ("mb_sample_off", "mb_samples", "mb_tokens", "mb_lmax", "mb_residual", "mb_cost", "mb_bucket", "mb_rank",
             "rank_mb_off", "rank_mbs", "sample_cost", "sample_mb")


def _gpu():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    import gpu_harness
    return gpu_harness


def oracle_from_device_sources(w, srcs, table):
    """Runs the oracle on host copies of the very source tensors the device used (the generator is the same
    code on both devices; test_generator_is_device_independent checks that separately)."""
    pool = OraclePool(PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    res = {"rc": []}
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        res["rc"].append(pool.register_samples(*register_args(w, samples)))
        res["rc"].append(pool.write_embeddings(*write_args(w, call), [srcs[c] for c in call], w.src_dtype))
    rc, plan = pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), PlanConfig(**plan_config_fields(w)))
    res["rc"].append(rc)
    res["plan"] = plan.arrays()
    n_mb, total, _ = plan.summary()
    out = np.full((total, w.hidden), 0xFFFF, dtype=np.uint16)
    cu = np.full(len(w.plan_order) + n_mb, -1, dtype=np.int32)
    pos = np.full(total, -1, dtype=np.int32)
    res["rc"].append(pool.gather_packed(plan, 0, n_mb, table, out, cu, pos))
    res.update(out=out, cu_seqlens=cu, position_ids=pos, status=pool.status())
    res["span_pages"] = {(s, j): pool.span_pages(s, j)[1] for call in w.write_calls for s, j in call}
    plan.destroy()
    pool.destroy()
    return res


def assert_same(got, exp):
    assert got["rc"] == exp["rc"]
    for k in PLAN_KEYS:
        assert np.array_equal(got["plan"][k], exp["plan"][k]), k
    assert got["plan"]["n_mb"] == exp["plan"]["n_mb"]
    for key, pages in exp["span_pages"].items():
        assert np.array_equal(got["span_pages"][key], pages), key   # same page assignment as the oracle's ring
    assert np.array_equal(got["cu_seqlens"], exp["cu_seqlens"])
    assert np.array_equal(got["position_ids"], exp["position_ids"])
    assert got["out"].shape == exp["out"].shape
    assert np.array_equal(got["out"], exp["out"])
    assert got["status"] == exp["status"]


CASES = [
    # name, kwargs, caller-owned memory            -- what the case stresses
    ("tiny", dict(), False),                                                  # config 1 at full size
    ("tiny", dict(hidden=64, page_bytes=4096), True),                         # caller-owned poisoned HBM
    ("image_mix_7b", dict(n_samples=14), False),                              # 7168 B rows straddle 2 MiB pages; host tier
    ("image_mix_7b", dict(n_samples=40, hidden=56, page_bytes=4096), False),  # 112 B rows, many pages per span, host tier
    ("image_mix_7b", dict(n_samples=10, hidden=4096, page_bytes=4096, all_hbm=True), False),  # 8 KiB rows over 4 KiB pages
    ("video_heavy", dict(n_samples=6), False),                                # 64 spans per sample, random write order
    ("host_tier_stress", dict(n_samples=3), False),                           # fp32 source + cast, shuffled ring, 50/50 tiers
    ("host_tier_stress", dict(n_samples=5, hidden=8192, page_bytes=4096), False),  # 16 KiB rows = 4-5 pages per row
]


@pytest.mark.parametrize("name,kw,owned", CASES)
def test_write_plan_gather_match_oracle(name, kw, owned):
    gh = _gpu()
    w = workloads.make_workload(name, **kw)
    got = gh.run_cuda(w, caller_owned_memory=owned)
    exp = oracle_from_device_sources(w, got["srcs"], got["table"])
    assert all(c == 0 for c in exp["rc"])
    assert_same(got, exp)
    assert not np.any(np.all(got["out"] == 0xFFFF, axis=1))  # every output row written
    assert got["stats"]["gpu_launches"] > 0


def test_generator_is_device_independent():
    _gpu()
    w = workloads.make_workload("host_tier_stress", n_samples=2, hidden=256)
    for s, j in [(0, 0), (1, 0)]:
        a = workloads.span_values(w, s, j, device="cpu")
        b = workloads.span_values(w, s, j, device="cuda").cpu()
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    w = workloads.make_workload("tiny")
    a = workloads.span_values(w, 3, 0, device="cpu")
    b = workloads.span_values(w, 3, 0, device="cuda").cpu()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    ta = workloads.embed_table(w, "cpu", rows=(100, 140))
    tb = workloads.embed_table(w, "cuda", rows=(100, 140)).cpu()
    assert torch.equal(ta.view(torch.int16), tb.view(torch.int16))


def test_cast_special_values_on_device():
    """Every special bit pattern through the fused cast equals the oracle's rule, NaNs included."""
    gh = _gpu()
    from paper_2606_23087_b200 import binding as fp
    bits = np.concatenate([workloads.special_f32_bits(), np.arange(0x3F7FF000, 0x3F801000, 1, dtype=np.uint32),
                           np.random.default_rng(7).integers(0, 1 << 32, 200000, dtype=np.uint64).astype(np.uint32)])
    H = 64
    n_tok = len(bits) // H
    bits = bits[:n_tok * H]
    src = torch.from_numpy(bits.view(np.int32).copy()).cuda()
    cfg = fp.PoolConfig(page_bytes=4096, hbm_pages=n_tok * 2 * H // 4096 + 2, host_pages=0, hidden=H, max_samples=1,
                        max_spans_per_sample=1, max_pages_per_span=1 << 16, max_seq_len=n_tok, max_text_tokens=n_tok + 1024,
                        placeholder_id=7)
    pool = fp.Pool(cfg)
    assert pool.rc == 0
    ids = torch.full((n_tok,), 7, dtype=torch.int32, device="cuda")
    assert pool.register_samples([0], [n_tok], [1], [0], [n_tok], ids.data_ptr(), gh.cuda_stream()) == 0
    assert pool.write_embeddings([0], [0], [n_tok], [src.data_ptr()], fp.FT_F32, gh.cuda_stream()) == 0
    rc, plan = pool.plan_microbatches([0], fp.PlanConfig(coef_A=1, coef_B=1, budget_L=n_tok, n_buckets_K=1, n_ranks_N=1))
    assert rc == 0
    out = torch.zeros((n_tok, H), dtype=torch.int16, device="cuda")
    cu = torch.zeros(2, dtype=torch.int32, device="cuda")
    pos = torch.zeros(n_tok, dtype=torch.int32, device="cuda")
    table = torch.zeros((8, H), dtype=torch.bfloat16, device="cuda")
    assert pool.gather_packed(plan, 0, 1, table.data_ptr(), 8, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream()) == 0
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint16).ravel()
    exp = np.array([f32_to_bf16_rne(int(b)) for b in bits], dtype=np.uint16)
    assert np.array_equal(got, exp)
    assert pool.status() == (0, 0)
    plan.destroy()
    pool.destroy()


def test_translate_matches_oracle():
    _gpu()
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("image_mix_7b", n_samples=6, hidden=64, page_bytes=4096)
    f = pool_config_fields(w)
    opool = OraclePool(PoolConfig(**f))
    pool = fp.Pool(fp.PoolConfig(**f))
    assert pool.rc == 0 and opool.rc == 0
    P = w.hbm_pages + w.host_pages
    gvas = [opool.page_gva(g) + d for g in range(P) for d in (0, 16, 4095)]
    gvas += [0, (1 << 44) - 1, (1 << 44) + w.hbm_pages * 4096, (1 << 44) + w.hbm_pages * 4096 + 4096 * 3 + 5,
             (1 << 45) - 1, (1 << 45) + w.host_pages * 4096, (1 << 45) + (1 << 40), (1 << 44) + (1 << 40) - 1, (1 << 63)]
    st, kind, frame, off = pool.translate(gvas)
    for i, g in enumerate(gvas):
        rc, k, fr, o = opool.translate(g)
        assert st[i] == rc, hex(g)
        if rc == 0:
            assert (int(kind[i]), int(frame[i]), int(off[i])) == (k, fr, o), hex(g)
    assert np.array_equal(pool.ring(), opool.ring())
    pool.destroy()
    opool.destroy()


def test_status_codes_match_oracle_call_by_call():
    gh = _gpu()
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("image_mix_7b", n_samples=6, hidden=64, page_bytes=4096)
    f = pool_config_fields(w)
    f["hbm_pages"], f["host_pages"] = w.pages_of_span(w.spans_of(0)[1][0]) + 1, 0
    opool, pool = OraclePool(PoolConfig(**f)), fp.Pool(fp.PoolConfig(**f))
    keep = []

    def both_register(samples=None, raw=None):
        a = register_args(w, samples) if raw is None else raw
        ids = torch.from_numpy(np.ascontiguousarray(a[5], dtype=np.int32)).cuda()
        keep.append(ids)
        g = pool.register_samples(*a[:5], ids.data_ptr(), gh.cuda_stream())
        o = opool.register_samples(*a)
        assert g == o, (g, o)
        return g

    def both_write(call, n_tokens=None):
        slots = np.array([s for s, _ in call], dtype=np.uint32)
        span_idx = np.array([j for _, j in call], dtype=np.uint32)
        real = [(s, j if j < int(w.n_spans[s]) else 0) for s, j in call]   # a source that exists, even for a bad index
        ntok = np.asarray([w.spans_of(s)[1][j] for s, j in real] if n_tokens is None else n_tokens, dtype=np.uint32)
        srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in real]
        keep.append(srcs)
        g = pool.write_embeddings(slots, span_idx, ntok, [t.data_ptr() for t in srcs], 0, gh.cuda_stream())
        o = opool.write_embeddings(slots, span_idx, ntok, [bits16(t) for t in srcs], 0)
        assert g == o, (g, o)
        return g

    def both_plan(slots, **kw):
        c = dict(coef_A=1, coef_B=1, budget_L=1 << 19, n_buckets_K=1, n_ranks_N=1, flags=0)
        c.update(kw)
        g, gp = pool.plan_microbatches(slots, fp.PlanConfig(**c), gh.cuda_stream())
        o, op = opool.plan_microbatches(slots, PlanConfig(**c))
        assert g == o, (g, o)
        return g, gp, op

    def both_free(slots):
        g, o = pool.free(slots, gh.cuda_stream()), opool.free(slots)
        assert g == o, (g, o)
        return g

    z = np.zeros(10, np.int32)
    assert both_register([0, 1, 2]) == 0
    assert both_register([3, 1]) == -10
    assert both_register(raw=([9], [10], [0], [], [], z)) == -1
    assert both_register(raw=([4], [10], [1], [8], [5], z)) == -1
    assert both_register(raw=([4], [10], [2], [2, 3], [2, 2], z)) == -1
    assert both_register(raw=([4], [10], [5], [0] * 5, [1] * 5, z)) == -11
    assert both_register(raw=([4], [0], [0], [], [], z)) == -1
    t0 = int(w.spans_of(0)[1][0])
    assert both_write([(3, 0)]) == -3
    assert both_write([(0, 7)], n_tokens=[t0]) == -1
    assert both_write([(0, 0)], n_tokens=[t0 + 1]) == -1
    assert both_write([(0, 0), (0, 0)]) == -4
    big = [(1, j) for j in range(int(w.n_spans[1]))] + [(2, j) for j in range(int(w.n_spans[2]))] + [(0, 0)]
    assert both_write(big) == -2
    assert pool.stats()["pages_free"] == opool.free_pages()[0] == f["hbm_pages"]
    assert both_write([(0, 0)]) == 0
    assert both_write([(0, 0)]) == -4
    assert both_plan([1])[0] == -5
    assert both_plan([5])[0] == -3
    assert both_plan([1, 1], flags=1)[0] == -1
    assert both_plan([1], flags=1, budget_L=10)[0] == -6
    assert both_plan([1], n_buckets_K=0)[0] == -1
    assert both_plan([1], coef_A=1 << 63, coef_B=1 << 40)[0] == -1
    rc, gp, op = both_plan([1, 2], flags=1)
    assert rc == 0 and gp.summary() == op.summary()
    total = gp.summary()[1]
    out = torch.zeros((total, 64), dtype=torch.int16, device="cuda")
    cu = torch.zeros(4, dtype=torch.int32, device="cuda")
    pos = torch.zeros(total, dtype=torch.int32, device="cuda")
    table = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    g = pool.gather_packed(gp, 0, 1, table.data_ptr(), 4, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream())
    o = opool.gather_packed(op, 0, 1, np.zeros((4, 64), np.uint16), np.zeros((total, 64), np.uint16), np.zeros(4, np.int32), np.zeros(total, np.int32))
    assert g == o == -5
    assert pool.gather_packed(gp, 1, 0, table.data_ptr(), 4, out.data_ptr(), cu.data_ptr(), pos.data_ptr()) == -1
    assert pool.gather_packed(gp, 0, 2, table.data_ptr(), 4, out.data_ptr(), cu.data_ptr(), pos.data_ptr()) == -1
    assert both_free([5]) == -3
    assert both_free([0, 0]) == -3
    assert both_free([0, 1, 2]) == 0
    assert pool.stats()["pages_free"] == opool.free_pages()[0]
    assert pool.stats()["text_pages_free"] == opool.free_pages()[1]
    assert np.array_equal(pool.ring(), opool.ring())
    assert pool.status() == opool.status() == (0, 0)
    pool.destroy()
    opool.destroy()


def test_async_errors_match_oracle():
    gh = _gpu()
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("tiny", n_samples=4, hidden=64, page_bytes=4096)
    f = pool_config_fields(w)
    opool, pool = OraclePool(PoolConfig(**f)), fp.Pool(fp.PoolConfig(**f))
    slots, seq_len, n_spans, pos, tok, ids = register_args(w, [0, 1, 2, 3])
    off = [0] + [int(x) for x in np.cumsum(seq_len)]
    ids = ids.copy()
    ids[off[2] + int(pos[2])] = 5
    text_pos = 0 if pos[1] > 0 else int(pos[1] + tok[1])
    ids[off[1] + text_pos] = w.placeholder_id
    d_ids = torch.from_numpy(ids).cuda()
    assert pool.register_samples(slots, seq_len, n_spans, pos, tok, d_ids.data_ptr(), gh.cuda_stream()) == 0
    assert opool.register_samples(slots, seq_len, n_spans, pos, tok, ids) == 0
    assert pool.status() == opool.status() == (-8, 1)
    assert pool.status() == (0, 0)
    assert pool.free([0, 1, 2, 3]) == opool.free([0, 1, 2, 3]) == 0
    # a token id outside the table: row skipped, smallest row index reported
    a = register_args(w, [0, 1])
    d_ids = torch.from_numpy(a[5]).cuda()
    assert pool.register_samples(*a[:5], d_ids.data_ptr(), gh.cuda_stream()) == opool.register_samples(*a) == 0
    call = [(0, 0), (1, 0)]
    srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]
    assert pool.write_embeddings(*write_args(w, call), [t.data_ptr() for t in srcs], 0, gh.cuda_stream()) == 0
    assert opool.write_embeddings(*write_args(w, call), [bits16(t) for t in srcs], 0) == 0
    cfg = dict(coef_A=1, coef_B=1, budget_L=4096, n_buckets_K=1, n_ranks_N=1, flags=0)
    rc, gp = pool.plan_microbatches([0, 1], fp.PlanConfig(**cfg), gh.cuda_stream())
    rc2, op = opool.plan_microbatches([0, 1], PlanConfig(**cfg))
    total = gp.summary()[1]
    small_vocab = 100
    table = torch.zeros((small_vocab, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.full((total, 64), -1, dtype=torch.int16, device="cuda")
    cu = torch.zeros(3, dtype=torch.int32, device="cuda")
    posb = torch.zeros(total, dtype=torch.int32, device="cuda")
    assert pool.gather_packed(gp, 0, 1, table.data_ptr(), small_vocab, out.data_ptr(), cu.data_ptr(), posb.data_ptr(), gh.cuda_stream()) == 0
    oout = np.full((total, 64), 0xFFFF, np.uint16)
    assert opool.gather_packed(op, 0, 1, np.zeros((small_vocab, 64), np.uint16), oout, np.zeros(3, np.int32), np.zeros(total, np.int32)) == 0
    assert pool.status() == opool.status()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oout)
    pool.destroy()
    opool.destroy()


@pytest.mark.parametrize("page_bytes", [4096, 65536])
def test_churn_then_gather_matches_oracle(page_bytes):
    """Fragmentation sweep in miniature: admit / free cycles, then plan + gather the residents."""
    gh = _gpu()
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("frag_sweep", n_samples=400, hidden=256, page_bytes=page_bytes, pool_bytes=24 << 20)
    ops, residents = workloads.admit_free_schedule(w, cycles=4)
    assert len(ops) >= 7
    f = pool_config_fields(w)
    f["max_text_tokens"] = 1024 * 2 * 400
    opool, pool = OraclePool(PoolConfig(**f)), fp.Pool(fp.PoolConfig(**f))
    assert pool.rc == 0 and opool.rc == 0
    keep = []
    for kind, samples in ops:
        if kind == "admit":
            a = register_args(w, samples)
            d_ids = torch.from_numpy(a[5]).cuda()
            keep.append(d_ids)
            assert pool.register_samples(*a[:5], d_ids.data_ptr(), gh.cuda_stream()) == opool.register_samples(*a) == 0
            call = [(s, 0) for s in samples]
            srcs = [workloads.span_values(w, s, 0, device="cuda") for s in samples]
            keep.append(srcs)
            assert pool.write_embeddings(*write_args(w, call), [t.data_ptr() for t in srcs], 0, gh.cuda_stream()) == 0
            assert opool.write_embeddings(*write_args(w, call), [bits16(t) for t in srcs], 0) == 0
        else:
            assert pool.free(samples, gh.cuda_stream()) == opool.free(samples) == 0
        assert np.array_equal(pool.ring(), opool.ring())
        assert pool.stats()["pages_free"] == opool.free_pages()[0]
    for s in residents[::7]:
        assert np.array_equal(pool.span_pages(s, 0)[1], opool.span_pages(s, 0)[1])
    cfg = plan_config_fields(w)
    rc, gp = pool.plan_microbatches(residents, fp.PlanConfig(**cfg), gh.cuda_stream())
    rc2, op = opool.plan_microbatches(residents, PlanConfig(**cfg))
    assert rc == rc2 == 0
    ga, oa = gp.arrays(), op.arrays()
    for k in PLAN_KEYS:
        assert np.array_equal(ga[k], oa[k]), k
    n_mb, total, _ = gp.summary()
    table = workloads.embed_table(w, device="cuda")
    out = torch.full((total, w.hidden), -1, dtype=torch.int16, device="cuda")
    cu = torch.full((len(residents) + n_mb,), -1, dtype=torch.int32, device="cuda")
    pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
    # gather in two ranges to exercise range offsets
    mid = n_mb // 2
    ga_tok = int(ga["mb_tokens"][:mid].sum())
    ga_cu = int(ga["mb_sample_off"][mid]) + mid
    assert pool.gather_packed(gp, 0, mid, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream()) == 0
    assert pool.gather_packed(gp, mid, n_mb, table.data_ptr(), w.vocab, out.data_ptr() + ga_tok * w.row_bytes,
                              cu.data_ptr() + 4 * ga_cu, pos.data_ptr() + 4 * ga_tok, gh.cuda_stream()) == 0
    torch.cuda.synchronize()
    oout = np.full((total, w.hidden), 0xFFFF, np.uint16)
    ocu = np.full(len(residents) + n_mb, -1, np.int32)
    opos = np.full(total, -1, np.int32)
    assert opool.gather_packed(op, 0, n_mb, bits16(table), oout, ocu, opos) == 0
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oout)
    assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos)
    assert pool.status() == opool.status() == (0, 0)
    pool.destroy()
    opool.destroy()


def test_planner_scale_matches_oracle():
    """65 536 descriptors (metadata only): every plan array equals the oracle's Algorithm 1."""
    gh = _gpu()
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("frag_sweep", n_samples=65536, hidden=64, page_bytes=4096, pool_bytes=4096 * 16)
    f = pool_config_fields(w)
    pool = fp.Pool(fp.PoolConfig(**f))
    assert pool.rc == 0
    # ids are irrelevant to the plan: register with all-placeholder-consistent ids generated on the device
    samples = list(range(w.n_samples))
    slots, seq_len, n_spans, pos, tok, _ = register_args(w, samples[:1])
    seq_len, n_spans = w.seq_len.astype(np.uint32), w.n_spans.astype(np.uint32)
    off = np.concatenate([[0], np.cumsum(seq_len.astype(np.int64))])
    ids = torch.zeros(int(off[-1]), dtype=torch.int32, device="cuda")
    starts = torch.from_numpy(off[:-1] + w.span_pos.astype(np.int64)).cuda()
    lens = torch.from_numpy(w.span_tokens.astype(np.int64)).cuda()
    mark = torch.zeros(int(off[-1]) + 1, dtype=torch.int32, device="cuda")
    mark.index_add_(0, starts, torch.ones_like(starts, dtype=torch.int32))
    mark.index_add_(0, starts + lens, -torch.ones_like(starts, dtype=torch.int32))
    ids[torch.cumsum(mark[:-1], 0) > 0] = w.placeholder_id
    assert pool.register_samples(samples, seq_len, n_spans, w.span_pos, w.span_tokens, ids.data_ptr(), gh.cuda_stream()) == 0
    assert pool.status() == (0, 0)
    order = [int(x) for x in np.random.default_rng(3).permutation(w.n_samples)]
    cfg = plan_config_fields(w, flags=1)
    rc, gp = pool.plan_microbatches(order, fp.PlanConfig(**cfg), gh.cuda_stream())
    assert rc == 0
    rc, op = plan_from_lengths(seq_len[order], PlanConfig(**cfg), slots=order)
    assert rc == 0
    ga, oa = gp.arrays(), op.arrays()
    assert ga["n_mb"] == oa["n_mb"] > 1000
    for k in PLAN_KEYS:
        assert np.array_equal(ga[k], oa[k]), k
    gp.destroy()
    op.destroy()
    pool.destroy()


@pytest.mark.parametrize("n", [150, 300, 1500, 6000])
def test_best_fit_ties_match_oracle_in_every_packing_kernel(n):
    """Lengths from a handful of values, budget 1000: equal residuals all the time, so the tie-break (the microbatch
    changed most recently) decides most placements.  The sample counts put the bound on the microbatch count
    (2 sum(l)/L + 1) into the range of each of the four packing kernels: registers (up to 128 and up to 256 microbatches),
    shared-memory scan (up to 1024), bitmap descent with per-residual stacks (beyond)."""
    gh = _gpu()
    from paper_2606_23087_b200 import binding as fp
    rng = np.random.default_rng(n)
    seq_len = rng.choice(np.array([100, 200, 250, 300, 400, 500], dtype=np.uint32), size=n).astype(np.uint32)
    pool = fp.Pool(fp.PoolConfig(page_bytes=4096, hbm_pages=16, host_pages=0, hidden=64, max_samples=n, max_spans_per_sample=1,
                                 max_pages_per_span=1, max_seq_len=1000, max_text_tokens=1024 * n, placeholder_id=7, world_size=1))
    assert pool.rc == 0
    d_ids = torch.zeros(int(seq_len.sum()), dtype=torch.int32, device="cuda")
    z = np.zeros(0, np.uint32)
    assert pool.register_samples(list(range(n)), seq_len, np.zeros(n, np.uint32), z, z, d_ids.data_ptr(), gh.cuda_stream()) == 0
    order = [int(x) for x in rng.permutation(n)]
    for flags in (0, 2):
        cfg = dict(coef_A=1000, coef_B=1, budget_L=1000, n_buckets_K=4, n_ranks_N=8, flags=flags)
        rc, gp = pool.plan_microbatches(order, fp.PlanConfig(**cfg), gh.cuda_stream())
        rc2, op = plan_from_lengths(seq_len[order], PlanConfig(**cfg), slots=order)
        assert rc == rc2 == 0
        ga, oa = gp.arrays(), op.arrays()
        assert ga["n_mb"] == oa["n_mb"]
        for k in PLAN_KEYS:
            assert np.array_equal(ga[k], oa[k]), (k, n, flags)
        gp.destroy(); op.destroy()
    assert pool.status() == (0, 0)
    pool.destroy()


# (flag 1 = ALLOW_UNWRITTEN: such a plan carries no row words, so its assembly resolves every row the long way)
@pytest.mark.parametrize("flags", [2, 4, 8, 16, 2 | 4 | 8 | 16, 1, 1 | 2])
def test_plan_variants_match_oracle(flags):
    """Scheduler variants (longest-first packing, sum-of-squares cost, carried zig-zag): every plan array equals
    the oracle's, on 6000 descriptors (metadata only) and on a written batch whose gather follows the new order."""
    gh = _gpu()
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("frag_sweep", n_samples=6000, hidden=64, page_bytes=4096, pool_bytes=4096 * 16)
    pool = fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    seq_len, n_spans = w.seq_len.astype(np.uint32), w.n_spans.astype(np.uint32)
    off = np.concatenate([[0], np.cumsum(seq_len.astype(np.int64))])
    ids = np.zeros(int(off[-1]), np.int32)
    for s in range(w.n_samples):
        p0 = int(off[s]) + int(w.span_pos[s])
        ids[p0:p0 + int(w.span_tokens[s])] = w.placeholder_id
    d_ids = torch.from_numpy(ids).cuda()
    assert pool.register_samples(list(range(w.n_samples)), seq_len, n_spans, w.span_pos, w.span_tokens, d_ids.data_ptr(), gh.cuda_stream()) == 0
    order = [int(x) for x in np.random.default_rng(flags).permutation(w.n_samples)]
    for K, N, L in ((4, 8, 32768), (1, 3, 18000), (7, 5, 131072), (3, 4, 65536)):   # (each budget takes another packing kernel)
        cfg = dict(coef_A=L, coef_B=1, budget_L=L, n_buckets_K=K, n_ranks_N=N, flags=flags | 1)
        rc, gp = pool.plan_microbatches(order, fp.PlanConfig(**cfg), gh.cuda_stream())
        rc2, op = plan_from_lengths(seq_len[order], PlanConfig(**cfg), slots=order)
        assert rc == rc2 == 0
        ga, oa = gp.arrays(), op.arrays()
        assert ga["n_mb"] == oa["n_mb"]
        for k in PLAN_KEYS:
            assert np.array_equal(ga[k], oa[k]), (k, K, N, L)
        gp.destroy(); op.destroy()
    pool.destroy()
    # end to end with the variant: the gather must follow the variant's append order
    w = workloads.make_workload("image_mix_7b", n_samples=24, hidden=128, page_bytes=16384)
    w.budget_L = 20000
    opool, pool = OraclePool(PoolConfig(**pool_config_fields(w))), fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
    keep = []
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        a = register_args(w, samples)
        d = torch.from_numpy(a[5]).cuda(); keep.append(d)
        assert pool.register_samples(*a[:5], d.data_ptr(), gh.cuda_stream()) == opool.register_samples(*a) == 0
        srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]; keep.append(srcs)
        assert pool.write_embeddings(*write_args(w, call), [t.data_ptr() for t in srcs], 0, gh.cuda_stream()) == 0
        assert opool.write_embeddings(*write_args(w, call), [bits16(t) for t in srcs], 0) == 0
    cfg = plan_config_fields(w, flags=flags)
    rc, gp = pool.plan_microbatches(w.plan_order, fp.PlanConfig(**cfg), gh.cuda_stream())
    rc2, op = opool.plan_microbatches(w.plan_order, PlanConfig(**cfg))
    assert rc == rc2 == 0
    n_mb, total, _ = gp.summary()
    assert (n_mb, total) == op.summary()[:2]
    table = workloads.embed_table(w, device="cuda")
    out = torch.full((total, w.hidden), -1, dtype=torch.int16, device="cuda")
    cu = torch.full((w.n_samples + n_mb,), -1, dtype=torch.int32, device="cuda")
    pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
    assert pool.gather_packed(gp, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream()) == 0
    oout = np.full((total, w.hidden), 0xFFFF, np.uint16); ocu = np.full(w.n_samples + n_mb, -1, np.int32); opos = np.full(total, -1, np.int32)
    assert opool.gather_packed(op, 0, n_mb, bits16(table), oout, ocu, opos) == 0
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oout)
    assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos)
    pool.destroy(); opool.destroy()


@pytest.mark.parametrize("name,kw", [
    ("image_mix_7b", dict(n_samples=40, hidden=56, page_bytes=4096)),    # host tier, many small microbatches
    ("image_mix_7b", dict(n_samples=14)),                                # 2 MiB pages, both tiers
    ("video_heavy", dict(n_samples=6)),
])
def test_rank_lists_match_oracle(name, kw):
    """A rank assembles the microbatches dealt to it (Algorithm 1, lines 15-27) in one call."""
    gh = _gpu()
    w = workloads.make_workload(name, **kw)
    w.budget_L = int(w.seq_len.max())          # several microbatches
    r = gh.CudaRun(w)
    r.run_schedule()
    rc, plan = r.plan()
    assert rc == 0
    a = plan.arrays()
    n_mb = int(a["n_mb"])
    assert n_mb >= 3
    table = workloads.embed_table(w, device="cuda")
    pool = OraclePool(PoolConfig(**pool_config_fields(w)))
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        assert pool.register_samples(*register_args(w, samples)) == 0
        assert pool.write_embeddings(*write_args(w, call), [gh.host_bits(r.srcs[c]) for c in call], w.src_dtype) == 0
    rc, oplan = pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), PlanConfig(**plan_config_fields(w)))
    assert rc == 0 and np.array_equal(oplan.arrays()["rank_mbs"], a["rank_mbs"])
    tok = a["mb_tokens"].astype(np.int64)
    n_s = np.diff(a["mb_sample_off"].astype(np.int64))
    lists = [[int(j) for j in a["rank_mbs"][a["rank_mb_off"][k]:a["rank_mb_off"][k + 1]]] for k in range(w.n_ranks_N)]
    lists += [list(range(n_mb))[::-1], [1, 1, 0], [n_mb - 1]]
    for lst in lists:
        rows, n_cu = int(tok[lst].sum()) if lst else 0, int((n_s[lst] + 1).sum()) if lst else 0
        out = torch.full((max(rows, 1), w.hidden), -1, dtype=torch.int16, device="cuda")
        cu = torch.full((max(n_cu, 1),), -7, dtype=torch.int32, device="cuda")
        pos = torch.full((max(rows, 1),), -7, dtype=torch.int32, device="cuda")
        g = r.pool.gather_list(plan, lst, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream())
        oout = np.full((max(rows, 1), w.hidden), 0xFFFF, np.uint16)
        ocu = np.full(max(n_cu, 1), -7, np.int32)
        opos = np.full(max(rows, 1), -7, np.int32)
        o = pool.gather_list(oplan, lst, bits16(table), oout, ocu, opos)
        assert g == o == 0
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy().view(np.uint16), oout), lst
        assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos), lst
    # errors: no such microbatch; ids outside a short table (detail = row in the list's output); dead plan
    args = (table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream())
    assert r.pool.gather_list(plan, [0, n_mb], *args) == pool.gather_list(oplan, [0, n_mb], bits16(table), oout, ocu, opos) == -1
    lst = [2, 0]
    rows = int(tok[lst].sum())
    out = torch.full((rows, w.hidden), -1, dtype=torch.int16, device="cuda")
    cu = torch.zeros((int((n_s[lst] + 1).sum()),), dtype=torch.int32, device="cuda")
    pos = torch.zeros((rows,), dtype=torch.int32, device="cuda")
    assert r.pool.gather_list(plan, lst, table.data_ptr(), 100, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream()) == 0
    oout = np.full((rows, w.hidden), 0xFFFF, np.uint16)
    assert pool.gather_list(oplan, lst, bits16(table)[:100], oout, np.zeros(len(cu), np.int32), np.zeros(rows, np.int32)) == 0
    st_g, st_o = r.pool.status(), pool.status()
    assert st_g == st_o and st_g[0] == -9
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oout)          # skipped rows stay untouched on both sides
    first = int(a["mb_samples"][0])
    assert r.pool.free([first], gh.cuda_stream()) == pool.free([first]) == 0
    assert r.pool.gather_list(plan, [0], *args) == pool.gather_list(oplan, [0], bits16(table), oout, ocu, opos) == -5
    oplan.destroy(); pool.destroy()
    r.close()


def test_library_limits_at_their_edges():
    """The largest row the assembly accepts (hidden 18432 over 4 KiB pages: a row touches up to 10 pages), one
    column more (CAPACITY, nothing written), the largest budget the planner accepts (2^20 - 1) and one more."""
    gh = _gpu()
    fp = gh.fp
    w = workloads.make_workload("tiny", n_samples=3, hidden=18432, page_bytes=4096)
    got = gh.run_cuda(w)
    exp = oracle_from_device_sources(w, got["srcs"], got["table"])
    assert_same(got, exp)
    w2 = workloads.make_workload("tiny", n_samples=2, hidden=18440, page_bytes=4096)
    r = gh.CudaRun(w2)
    r.run_schedule()
    rc, plan = r.plan()
    assert rc == 0
    rc, out, cu, pos = r.gather_all(table=torch.zeros((w2.vocab, w2.hidden), dtype=torch.bfloat16, device="cuda"))
    assert rc == -11 and bool((out == -1).all().item())
    lst_rc = r.pool.gather_list(plan, [0], r.table.data_ptr(), w2.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), gh.cuda_stream())
    assert lst_rc == -11
    r.close()
    # planner budgets
    w3 = workloads.make_workload("tiny", n_samples=8, hidden=64, page_bytes=4096)
    r = gh.CudaRun(w3)
    r.run_schedule()
    lens = w3.seq_len[w3.plan_order]
    for L, want in (((1 << 20) - 1, 0), (1 << 20, -11)):
        cfg = dict(coef_A=3, coef_B=1, budget_L=L, n_buckets_K=2, n_ranks_N=3, flags=0)
        rc, gp = r.pool.plan_microbatches(np.asarray(w3.plan_order, np.uint32), fp.PlanConfig(**cfg), gh.cuda_stream())
        assert rc == want
        if rc == 0:
            rc2, op = plan_from_lengths(lens, PlanConfig(**cfg), slots=w3.plan_order)
            ga, oa = gp.arrays(), op.arrays()
            for k in PLAN_KEYS:
                assert np.array_equal(ga[k], oa[k]), k
            assert ga["n_mb"] == 1
            gp.destroy(); op.destroy()
    r.close()
