"""Differential test: a seeded random sequence of pool calls (valid and invalid) is fed to the CUDA library and
to the CPU oracle; every status code, the free ring after every mutating call, every plan array and every
gathered byte must agree."""
import numpy as np
import pytest
import torch

import workloads
from harness import bits16, pool_config_fields, register_args
from oracle import OraclePool, PlanConfig, PoolConfig

pytestmark = pytest.mark.gpu

PLAN_KEYS = ("mb_sample_off", "mb_samples", "mb_tokens", "mb_lmax", "mb_residual", "mb_cost", "mb_bucket", "mb_rank",
             "rank_mb_off", "rank_mbs", "sample_cost", "sample_mb")


# (copy_engine = 1: host-tier pages of writes and assemblies go through the copy engines, from the host's own copy of
# the page ring, which the churn of this test has to keep in step with the device's)
@pytest.mark.parametrize("seed,ring_order,page_bytes,hidden,copy_engine", [
    (0, 0, 4096, 64, 0), (1, 1, 4096, 56, 0), (2, 1, 16384, 1024, 0), (3, 1, 4096, 64, 1), (4, 0, 16384, 1024, 1)])
def test_random_call_sequences_agree_with_oracle(seed, ring_order, page_bytes, hidden, copy_engine):
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import cuda_stream
    from paper_2606_23087_b200 import binding as fp
    rng = np.random.default_rng(seed)
    w = workloads.make_workload("image_mix_7b", n_samples=48, hidden=hidden, page_bytes=page_bytes)
    w.ring_order = ring_order
    f = pool_config_fields(w)
    # a pool that holds roughly half of the samples, split over both tiers: exhaustion and host pages both occur
    need = sum(w.pages_of_span(t) for t in w.span_tokens)
    f["hbm_pages"], f["host_pages"] = need // 4, need // 4
    f["max_text_tokens"] = w.total_text_tokens_capacity // 2
    opool, pool = OraclePool(PoolConfig(**f)), fp.Pool(fp.PoolConfig(**f))
    assert pool.rc == 0 and opool.rc == 0
    assert pool.set_tuning(host_copy_engine=copy_engine) == 0
    table = workloads.embed_table(w, device="cuda")
    table_h = bits16(table)
    keep, plans = [], []
    n_calls = {"register": 0, "write": 0, "free": 0, "plan": 0, "gather": 0, "glist": 0, "grids": 0, "padded": 0, "grad": 0}
    n_ok = dict(n_calls)

    def check_state():
        assert np.array_equal(pool.ring(), opool.ring())
        st = pool.stats()
        assert (st["pages_free"], st["text_pages_free"]) == opool.free_pages()

    # a light model of the pool's state steers the generator toward calls that succeed most of the time;
    # whether a call did succeed is still decided by the two implementations alone
    state = {}      # slot -> set of written span indices

    def ready():
        return [s for s, wr in state.items() if len(wr) == int(w.n_spans[s])]

    for step in range(260):
        op = rng.choice(["register", "write", "write", "free", "plan", "gather", "glist", "grids", "padded", "grad"])
        n_calls[op] += 1
        sloppy = rng.random() < 0.2     # one call in five is built without looking at the model
        if op == "register":
            free_slots = [s for s in range(w.n_samples) if s not in state]
            if sloppy or not free_slots:
                samples = [min(int(x), w.n_samples - 1) for x in rng.choice(w.n_samples + 2, size=int(rng.integers(1, 6)))]
            else:
                samples = [int(x) for x in rng.choice(free_slots, size=min(len(free_slots), int(rng.integers(1, 5))), replace=False)]
            a = list(register_args(w, samples))
            if sloppy and rng.random() < 0.3:
                a[0] = a[0].copy(); a[0][0] = w.n_samples + 5          # slot out of range
            ids = torch.from_numpy(a[5]).cuda()
            keep.append(ids)
            g = pool.register_samples(*a[:5], ids.data_ptr(), cuda_stream())
            o = opool.register_samples(*a)
            if g == 0:
                for s_ in samples:
                    state[s_] = set()
        elif op == "write":
            todo = [(s_, j) for s_, wr in state.items() for j in range(int(w.n_spans[s_])) if j not in wr]
            if sloppy or not todo:
                k = int(rng.integers(1, 7))
                slots = rng.integers(0, w.n_samples, size=k)
                span_idx = np.array([rng.integers(0, int(w.n_spans[s_]) + (1 if rng.random() < 0.1 else 0)) for s_ in slots])
            else:
                pick = [todo[i] for i in rng.choice(len(todo), size=min(len(todo), int(rng.integers(1, 8))), replace=False)]
                slots = np.array([s_ for s_, _ in pick]); span_idx = np.array([j for _, j in pick])
            real = [(int(s_), int(min(j, int(w.n_spans[s_]) - 1))) for s_, j in zip(slots, span_idx)]
            ntok = np.array([int(w.spans_of(s_)[1][j]) + (1 if sloppy and rng.random() < 0.1 else 0) for s_, j in real], dtype=np.uint32)
            srcs = [workloads.span_values(w, s_, j, device="cuda") for s_, j in real]
            keep.append(srcs)
            g = pool.write_embeddings(slots, span_idx, ntok, [t.data_ptr() for t in srcs], 0, cuda_stream())
            o = opool.write_embeddings(slots, span_idx, ntok, [bits16(t) for t in srcs], 0)
            if g == 0:
                for s_, j in real:
                    state[s_].add(j)
        elif op == "free":
            if sloppy or not state:
                slots = rng.integers(0, w.n_samples, size=int(rng.integers(1, 5)))
            else:
                slots = rng.choice(list(state), size=min(len(state), int(rng.integers(1, 4))), replace=False)
            g, o = pool.free(slots, cuda_stream()), opool.free(slots)
            if g == 0:
                for s_ in slots:
                    state.pop(int(s_))
        elif op == "plan":
            rdy = ready()
            if sloppy or not rdy:
                slots = rng.choice(w.n_samples, size=int(rng.integers(0, 20)), replace=bool(rng.random() < 0.2))
                cfg = dict(coef_A=int(rng.integers(0, 50000)), coef_B=int(rng.integers(0, 3)),
                           budget_L=int(rng.choice([0, 6000, 20000, 40000, 1 << 19])), n_buckets_K=int(rng.integers(0, 5)),
                           n_ranks_N=int(rng.integers(0, 9)), flags=int(rng.random() < 0.5) + 2 * int(rng.integers(0, 16)))
            else:
                slots = rng.permutation(rdy)[:int(rng.integers(1, len(rdy) + 1))]
                cfg = dict(coef_A=int(rng.integers(0, 50000)), coef_B=int(rng.integers(0, 3)),
                           budget_L=int(rng.choice([w.max_seq_len, 20000, 40000, 1 << 19])), n_buckets_K=int(rng.integers(1, 5)),
                           n_ranks_N=int(rng.integers(1, 9)), flags=2 * int(rng.integers(0, 16)))
            g, gp = pool.plan_microbatches(slots, fp.PlanConfig(**cfg), cuda_stream())
            o, op_ = opool.plan_microbatches(slots, PlanConfig(**cfg))
            if g == 0 and o == 0:
                ga, oa = gp.arrays(), op_.arrays()
                assert ga["n_mb"] == oa["n_mb"]
                for key in PLAN_KEYS:
                    assert np.array_equal(ga[key], oa[key]), (step, key)
                plans.append((gp, op_, len(slots), cfg["budget_L"]))
                plans[:] = plans[-4:]
        elif op == "glist":
            if not plans:
                n_calls[op] -= 1
                continue
            gp, op_, n, _budget = plans[int(rng.integers(0, len(plans)))]
            n_mb, total, _ = op_.summary()
            oa_ = op_.arrays()
            lst = [int(x) for x in rng.integers(0, n_mb + (1 if sloppy else 0), size=int(rng.integers(0, 6)))] if n_mb or sloppy else []
            ok_l = [j for j in lst if j < n_mb]
            rows = max(1, int(sum(int(oa_["mb_tokens"][j]) for j in ok_l)))
            n_cu = max(1, int(sum(int(oa_["mb_sample_off"][j + 1] - oa_["mb_sample_off"][j]) + 1 for j in ok_l)))
            out = torch.full((rows, w.hidden), -1, dtype=torch.int16, device="cuda")
            cu = torch.full((n_cu,), -7, dtype=torch.int32, device="cuda")
            pos = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
            g = pool.gather_list(gp, lst, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), cuda_stream())
            oout = np.full((rows, w.hidden), 0xFFFF, np.uint16)
            ocu = np.full(n_cu, -7, np.int32)
            opos = np.full(rows, -7, np.int32)
            o = opool.gather_list(op_, lst, table_h, oout, ocu, opos)
            if g == 0 and o == 0:
                torch.cuda.synchronize()
                assert np.array_equal(out.cpu().numpy().view(np.uint16), oout), step
                assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos), step
        elif op == "grids":
            if sloppy or not state:
                k = int(rng.integers(1, 4))
                slots = rng.integers(0, w.n_samples + 1, size=k)
                spans = rng.integers(0, 5, size=k)
                grids = rng.integers(0, 40, size=(k, 3))
            else:
                slots = rng.choice(list(state.keys()), size=int(rng.integers(1, 4)))
                spans = [int(rng.integers(0, int(w.n_spans[s_]))) for s_ in slots]
                grids = []
                for s_, j_ in zip(slots, spans):
                    n_tok = int(w.spans_of(int(s_))[1][j_])
                    d = [x for x in range(1, 65) if n_tok % x == 0]
                    wdt = int(rng.choice(d))
                    t_ = int(rng.choice([x for x in (1, 2, 3) if (n_tok // wdt) % x == 0]))
                    grids.append([t_, n_tok // wdt // t_, wdt])
            g, o = pool.set_span_grids(slots, spans, grids, cuda_stream()), opool.set_span_grids(slots, spans, grids)
        elif op in ("padded", "grad"):
            if not plans:
                n_calls[op] -= 1
                continue
            gp, op_, n, budget = plans[int(rng.integers(0, len(plans)))]
            n_mb, total, _ = op_.summary()
            lo = int(rng.integers(0, n_mb + 1))
            hi = int(rng.integers(0, n_mb + 2))
            padded_layout = op == "padded" or bool(rng.random() < 0.5)
            rows = max(1, (max(hi - lo, 0) * budget) if padded_layout else int(total))
            if rows * w.hidden > (96 << 20):   # keep the buffers of one call below a few hundred MB
                n_calls[op] -= 1
                continue
            if op == "padded":
                out = torch.full((rows, w.hidden), -1, dtype=torch.int16, device="cuda")
                cu = torch.full((n + 2 * n_mb + 2,), -7, dtype=torch.int32, device="cuda")
                pos3 = torch.full((3, rows), -7, dtype=torch.int32, device="cuda")
                ids_, lab = (torch.full((rows,), -7, dtype=torch.int32, device="cuda") for _ in range(2))
                msk = torch.full((rows,), 7, dtype=torch.uint8, device="cuda")
                g = pool.gather_padded(gp, lo, hi, table.data_ptr(), w.vocab, -1, out.data_ptr(), cu.data_ptr(), pos3.data_ptr(),
                                       ids_.data_ptr(), lab.data_ptr(), msk.data_ptr(), cuda_stream())
                eo = dict(out=np.full((rows, w.hidden), 0xFFFF, np.uint16), cu=np.full(n + 2 * n_mb + 2, -7, np.int32),
                          pos3=np.full((3, rows), -7, np.int32), ids=np.full(rows, -7, np.int32), labels=np.full(rows, -7, np.int32),
                          mask=np.full(rows, 7, np.uint8))
                o = opool.gather_padded(op_, lo, hi, table_h, -1, eo["out"], eo["cu"], eo["pos3"], eo["ids"], eo["labels"], eo["mask"])
                if g == 0 and o == 0:
                    torch.cuda.synchronize()
                    if hi > lo:   # an empty range writes nothing; the layouts of the poison differ ([3, rows] with rows = 1)
                        got = dict(out=out.cpu().numpy().view(np.uint16), cu=cu.cpu().numpy(), pos3=pos3.cpu().numpy(),
                                   ids=ids_.cpu().numpy(), labels=lab.cpu().numpy(), mask=msk.cpu().numpy())
                        for key in got:
                            assert np.array_equal(got[key], eo[key]), (step, key)
            else:
                grad = workloads.grad_values(w, 0, rows, device="cuda")
                gt = torch.zeros((w.vocab, w.hidden), dtype=torch.float32, device="cuda")
                g = pool.embed_grad(gp, lo, hi, padded_layout, grad.data_ptr(), gt.data_ptr(), w.vocab, cuda_stream())
                et = np.zeros((w.vocab, w.hidden), np.float32)
                o = opool.embed_grad(op_, lo, hi, padded_layout, bits16(grad), et)
                if g == 0 and o == 0:
                    torch.cuda.synchronize()
                    assert np.array_equal(gt.cpu().numpy().view(np.uint32), et.view(np.uint32)), step
        else:
            if not plans:
                continue
            gp, op_, n, _budget = plans[int(rng.integers(0, len(plans)))]
            n_mb, total, _ = op_.summary()
            lo = int(rng.integers(0, n_mb + 1))
            hi = int(rng.integers(0, n_mb + 2))
            rows = max(1, int(total))
            out = torch.full((rows, w.hidden), -1, dtype=torch.int16, device="cuda")
            cu = torch.full((n + n_mb + 2,), -7, dtype=torch.int32, device="cuda")
            pos = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
            g = pool.gather_packed(gp, lo, hi, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(),
                                   cuda_stream())
            oout = np.full((rows, w.hidden), 0xFFFF, np.uint16)
            ocu = np.full(n + n_mb + 2, -7, np.int32)
            opos = np.full(rows, -7, np.int32)
            o = opool.gather_packed(op_, lo, hi, table_h, oout, ocu, opos)
            if g == 0 and o == 0:
                torch.cuda.synchronize()
                assert np.array_equal(out.cpu().numpy().view(np.uint16), oout), step
                assert np.array_equal(cu.cpu().numpy(), ocu) and np.array_equal(pos.cpu().numpy(), opos), step
        assert g == o, (step, op, g, o)
        if g == 0:
            n_ok[op] += 1
        if op in ("register", "write", "free"):
            check_state()
    assert pool.status() == opool.status()
    # the sequence must have exercised successes and failures of every call
    for k in n_calls:
        assert 0 < n_ok[k] <= n_calls[k], (k, n_ok, n_calls)
    assert any(n_ok[k] < n_calls[k] for k in n_calls)
    pool.destroy()
    opool.destroy()
