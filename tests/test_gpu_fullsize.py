"""Parity at the sizes the five configurations name, in the launch configuration bench.py times.

The plan is compared array by array with the oracle's Algorithm 1 on the same lengths; cu_seqlens and position
ids are compared in full with what the plan arrays determine; and EVERY assembled row is compared, on the device,
with the row the consumer semantics fix (Sec. 3.1-3.2: a placeholder position reads the span's row through its
GVA, any other position the table row of its id), rebuilt sample by sample from the seeded generator with plain
tensor indexing -- no library call on that side.  Where the host has the memory for it, the oracle itself also
runs once at full size and its whole output is compared.  Sampled rows are still checked one by one against rows
the oracle side computes (for fp32 sources through the oracle's own cast)."""
import gc
import numpy as np
import pytest
import torch

import workloads
from harness import bits16, bits32, plan_config_fields
from oracle import PlanConfig, f32_to_bf16_rne, plan_from_lengths

pytestmark = pytest.mark.gpu

def rne_bf16_bits(x_f32):
    """bf16 bit patterns (int16 tensor) of an fp32 tensor under the write path's rule, in integer arithmetic on
    the device: round to nearest even on the bit pattern, denormals kept, every NaN -> sign | 0x7FC0.  A test-side
    restatement used only to cover 100 % of rows at sizes the oracle cannot hold; test_cast_restatement_equals_oracle
    ties it to the oracle's cast."""
    u = x_f32.contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    r = torch.where(nan, ((u >> 16) & 0x8000) | 0x7FC0, r) & 0xFFFF
    return torch.where(r >= 0x8000, r - 0x10000, r).to(torch.int16)


def expected_sample_rows(w, s, table_i16):
    """int16 [seq_len, H] on the device: what the assembly of sample s must contain, from the generator alone."""
    ids = torch.from_numpy(workloads.input_ids(w, s).astype(np.int64)).cuda()
    exp = table_i16[ids]                       # text rows (rows at placeholder positions are overwritten below)
    pos, tok = w.spans_of(s)
    for j in range(len(pos)):
        v = workloads.span_values(w, s, j, device="cuda")
        v = v.view(torch.int16) if w.src_dtype == 0 else rne_bf16_bits(v)
        exp[int(pos[j]):int(pos[j]) + int(tok[j])] = v
    return exp


def assert_every_row(w, out_i16, samples, row_offsets, table_i16):
    """Compares all rows of `out_i16` that belong to the listed samples (sample k starts at row_offsets[k])."""
    bad = []
    for k, s in enumerate(samples):
        exp = expected_sample_rows(w, int(s), table_i16)
        r0 = int(row_offsets[k])
        if not torch.equal(out_i16[r0:r0 + exp.shape[0]], exp):
            bad.append(int(s))
    assert not bad, f"{len(bad)} samples differ, first {bad[:5]}"
    return len(samples)


def host_mem_available():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def oracle_full_output(w, srcs_dev, table_dev):
    """The oracle itself on the whole workload (host copies of the very tensors the device read):
    (plan arrays, out uint16 [rows, H], cu, pos)."""
    from harness import pool_config_fields, register_args, write_args
    from gpu_harness import host_bits
    from oracle import OraclePool, PoolConfig
    pool = OraclePool(PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        assert pool.register_samples(*register_args(w, samples)) == 0
        assert pool.write_embeddings(*write_args(w, call), [host_bits(srcs_dev[c]) for c in call], w.src_dtype) == 0
    rc, plan = pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), PlanConfig(**plan_config_fields(w)))
    assert rc == 0
    n_mb, total, _ = plan.summary()
    out = np.full((total, w.hidden), 0xFFFF, dtype=np.uint16)
    cu = np.full(len(w.plan_order) + n_mb, -1, dtype=np.int32)
    pos = np.full(total, -1, dtype=np.int32)
    assert pool.gather_packed(plan, 0, n_mb, bits16(table_dev), out, cu, pos) == 0
    assert pool.status() == (0, 0)
    plan.destroy()
    pool.destroy()
    return out, cu, pos


PLAN_KEYS = ("mb_sample_off", "mb_samples", "mb_tokens", "mb_lmax", "mb_residual", "mb_cost", "mb_bucket", "mb_rank",
             "rank_mb_off", "rank_mbs", "sample_cost", "sample_mb")


def expected_row(w, s, p):
    """Row of position p of sample s, from the generator (oracle side; no CUDA library involved)."""
    pos, tok = w.spans_of(s)
    for j in range(len(pos)):
        if int(pos[j]) <= p < int(pos[j]) + int(tok[j]):
            r = p - int(pos[j])
            v = workloads.span_values(w, s, j, device="cpu", rows=(r, r + 1))
            if w.src_dtype == 0:
                return bits16(v).ravel()
            return np.array([f32_to_bf16_rne(int(b)) for b in bits32(v).ravel()], dtype=np.uint16)
    i = int(workloads.input_ids(w, s)[p])
    return bits16(workloads.embed_table(w, "cpu", rows=(i, i + 1))).ravel()


FULL_ORACLE = {}


def test_cast_restatement_equals_oracle():
    """The integer restatement of the cast that the full-coverage compare uses for fp32 sources, against the oracle:
    a whole sample of the host-tier-stress workload (special bit patterns included) written and assembled by the
    oracle, and every special pattern through the oracle's scalar cast."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from harness import host_span, pool_config_fields
    from oracle import OraclePool, PoolConfig
    spec = workloads.special_f32_bits()
    t = torch.from_numpy(spec.view(np.int32).copy()).cuda().view(torch.float32)
    assert np.array_equal(rne_bf16_bits(t).cpu().numpy().view(np.uint16),
                          np.array([f32_to_bf16_rne(int(b)) for b in spec], dtype=np.uint16))
    w = workloads.make_workload("host_tier_stress", n_samples=3)
    table = workloads.embed_table(w, device="cuda")
    for s in (0, 2):
        f = pool_config_fields(w, max_samples=1)
        f.update(hbm_pages=w.pages_of_span(int(w.spans_of(s)[1][0])) + 1, host_pages=0)
        pool = OraclePool(PoolConfig(**f))
        assert pool.rc == 0
        pos, tok = w.spans_of(s)
        assert pool.register_samples([0], [int(w.seq_len[s])], [1], pos, tok, workloads.input_ids(w, s)) == 0
        assert pool.write_embeddings([0], [0], tok, [host_span(w, s, 0)], 1) == 0
        rc, plan = pool.plan_microbatches([0], PlanConfig(**plan_config_fields(w)))
        assert rc == 0
        n = int(w.seq_len[s])
        out = np.zeros((n, w.hidden), np.uint16)
        assert pool.gather_packed(plan, 0, 1, bits16(table), out, np.zeros(2, np.int32), np.zeros(n, np.int32)) == 0
        exp = expected_sample_rows(w, s, table.view(torch.int16)).cpu().numpy().view(np.uint16)
        assert np.array_equal(out, exp)
        plan.destroy(); pool.destroy()


@pytest.mark.parametrize("name,kw", [("image_mix_7b", {}), ("video_heavy", {}), ("host_tier_stress", {})])
def test_full_size_plan_and_sampled_rows(name, kw):
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import CudaRun
    w = workloads.make_workload(name, **kw)
    run = CudaRun(w)
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        assert run.register(samples) == 0
        assert run.write(call, keep_src=True) == 0
    rc, plan = run.plan()
    assert rc == 0
    got = plan.arrays()
    rc, oplan = plan_from_lengths(w.seq_len[w.plan_order], PlanConfig(**plan_config_fields(w)), slots=w.plan_order)
    assert rc == 0
    exp = oplan.arrays()
    for k in PLAN_KEYS:
        assert np.array_equal(got[k], exp[k]), k
    assert plan.summary() == oplan.summary()
    rc, out, cu, pos = run.gather_all()
    assert rc == 0 and run.pool.status() == (0, 0)
    # what the plan arrays determine about cu_seqlens / position ids (numpy only)
    lens = w.seq_len[exp["mb_samples"]].astype(np.int64)
    exp_pos = np.concatenate([np.arange(l, dtype=np.int32) for l in lens])
    assert np.array_equal(pos.cpu().numpy(), exp_pos)
    exp_cu = []
    for j in range(exp["n_mb"]):
        a, b = int(exp["mb_sample_off"][j]), int(exp["mb_sample_off"][j + 1])
        exp_cu.append(np.concatenate([[0], np.cumsum(lens[a:b])]))
    assert np.array_equal(cu.cpu().numpy(), np.concatenate(exp_cu).astype(np.int32))
    # sampled rows, including each sample's first/last rows and span boundaries
    row_off = np.concatenate([[0], np.cumsum(lens)])
    rng = np.random.default_rng(11)
    picks = []
    for q in rng.choice(len(lens), size=24, replace=False):
        s = int(exp["mb_samples"][q])
        sp, st = w.spans_of(s)
        cand = {0, int(lens[q]) - 1, int(rng.integers(0, lens[q]))}
        j = int(rng.integers(0, len(sp)))
        cand |= {int(sp[j]), int(sp[j]) + int(st[j]) - 1, min(int(lens[q]) - 1, int(sp[j]) + int(st[j]))}
        if int(sp[j]) > 0:
            cand.add(int(sp[j]) - 1)
        picks += [(q, s, p) for p in sorted(cand)]
    rows = torch.tensor([int(row_off[q]) + p for q, s, p in picks], device="cuda")
    got_rows = out[rows].cpu().numpy().view(np.uint16)
    for i, (q, s, p) in enumerate(picks):
        exp_row = expected_row(w, s, p)
        assert np.array_equal(got_rows[i], exp_row), (q, s, p)
        if w.src_dtype == 1:   # the special bit patterns (every 4099th element) reach some sampled rows
            pass
    # no row left at poison anywhere (checked on the device)
    assert not bool((out == -1).all(dim=1).any().item())
    # EVERY row of the assembly against the generator (device-side compare, sample by sample)
    table_i16 = run.table.view(torch.int16)
    assert assert_every_row(w, out, exp["mb_samples"], row_off[:-1], table_i16) == w.n_samples
    assert int(row_off[-1]) == out.shape[0]
    # the oracle itself at full size, whole output, where the host can hold its pool, the sources and the result
    src_bytes = sum(t.numel() * t.element_size() for t in run.srcs.values())
    need = src_bytes + (w.hbm_pages + w.host_pages) * w.page_bytes + 2 * out.numel() * 2 + (4 << 30)
    FULL_ORACLE[name] = False
    if w.src_dtype == 0 and host_mem_available() >= int(1.25 * need):
        o_out, o_cu, o_pos = oracle_full_output(w, run.srcs, run.table)
        assert np.array_equal(o_cu, cu.cpu().numpy()) and np.array_equal(o_pos, pos.cpu().numpy())
        step = 1 << 18
        for r in range(0, out.shape[0], step):
            assert np.array_equal(out[r:r + step].cpu().numpy().view(np.uint16), o_out[r:r + step]), r
        del o_out
        FULL_ORACLE[name] = True
    print(f"full-size {name}: all {out.shape[0]} rows equal the generator's; whole-output oracle run: {FULL_ORACLE[name]}")
    # every rank's share of the deal in one list call each: the same rows, cu_seqlens and positions as the
    # slices of the range assembly checked above
    from gpu_harness import cuda_stream
    mb_rows = np.concatenate([[0], np.cumsum(exp["mb_tokens"].astype(np.int64))])
    mb_cu = np.concatenate([[0], np.cumsum(np.diff(exp["mb_sample_off"].astype(np.int64)) + 1)])
    cu_h, pos_h = cu.cpu().numpy(), pos.cpu().numpy()
    cap = int(max(sum(mb_rows[j + 1] - mb_rows[j] for j in exp["rank_mbs"][exp["rank_mb_off"][k]:exp["rank_mb_off"][k + 1]])
                  for k in range(w.n_ranks_N)))
    l_out = torch.empty((cap, w.hidden), dtype=torch.int16, device="cuda")
    l_cu = torch.empty((len(cu_h),), dtype=torch.int32, device="cuda")
    l_pos = torch.empty((cap,), dtype=torch.int32, device="cuda")
    for k in range(w.n_ranks_N):
        lst = [int(j) for j in exp["rank_mbs"][exp["rank_mb_off"][k]:exp["rank_mb_off"][k + 1]]]
        if not lst:
            continue
        l_out.fill_(-1)
        assert run.pool.gather_list(plan, lst, run.table.data_ptr(), w.vocab, l_out.data_ptr(), l_cu.data_ptr(), l_pos.data_ptr(),
                                    cuda_stream()) == 0
        torch.cuda.synchronize()
        base = c_base = 0
        for j in lst:
            n_r, n_c = int(mb_rows[j + 1] - mb_rows[j]), int(mb_cu[j + 1] - mb_cu[j])
            assert torch.equal(l_out[base:base + n_r], out[int(mb_rows[j]):int(mb_rows[j + 1])])
            assert np.array_equal(l_pos[base:base + n_r].cpu().numpy(), pos_h[mb_rows[j]:mb_rows[j + 1]])
            assert np.array_equal(l_cu[c_base:c_base + n_c].cpu().numpy(), cu_h[mb_cu[j]:mb_cu[j + 1]])
            base += n_r; c_base += n_c
    assert run.pool.status() == (0, 0)
    oplan.destroy()
    run.close()


def _oracle_samples(w, samples):
    """Oracle pool holding only the given samples (slot k = k-th of them), written, gridded, planned together;
    returns per-sample (positions [3, n], ids, labels, mask) read from its padded assembly."""
    from harness import host_span, pool_config_fields
    from oracle import OraclePool, PoolConfig
    f = pool_config_fields(w, max_samples=len(samples))
    need = sum(w.pages_of_span(int(t)) for s in samples for t in w.spans_of(s)[1])
    f.update(hbm_pages=need + 2, host_pages=0, max_text_tokens=int(sum(int(w.seq_len[s]) for s in samples)) + 1024 * len(samples))
    pool = OraclePool(PoolConfig(**f))
    assert pool.rc == 0
    for k, s in enumerate(samples):
        pos, tok = w.spans_of(s)
        assert pool.register_samples([k], [int(w.seq_len[s])], [len(pos)], pos, tok, workloads.input_ids(w, s)) == 0
        if len(pos):
            assert pool.write_embeddings([k] * len(pos), list(range(len(pos))), tok, [host_span(w, s, j) for j in range(len(pos))], w.src_dtype) == 0
        items = [(j, workloads.span_grid(w, s, j)) for j in range(len(pos))]
        items = [it for it in items if it[1] is not None]
        assert pool.set_span_grids([k] * len(items), [j for j, _ in items], [g for _, g in items]) == 0
    cfg = plan_config_fields(w)
    rc, plan = pool.plan_microbatches(list(range(len(samples))), PlanConfig(**cfg))
    assert rc == 0
    a = plan.arrays()
    n_mb, L = int(a["n_mb"]), w.budget_L
    rows = n_mb * L
    o = dict(out=np.zeros((rows, w.hidden), np.uint16), cu=np.zeros(len(samples) + 2 * n_mb, np.int32), pos3=np.zeros((3, rows), np.int32),
             ids=np.zeros(rows, np.int32), labels=np.zeros(rows, np.int32), mask=np.zeros(rows, np.uint8))
    table = np.zeros((w.vocab, w.hidden), np.uint16)
    assert pool.gather_padded(plan, 0, n_mb, table, 0, o["out"], o["cu"], o["pos3"], o["ids"], o["labels"], o["mask"]) == 0
    res = {}
    for j in range(n_mb):
        row = j * L
        for k in a["mb_samples"][a["mb_sample_off"][j]:a["mb_sample_off"][j + 1]]:
            n = int(w.seq_len[samples[int(k)]])
            res[samples[int(k)]] = (o["pos3"][:, row:row + n].copy(), o["ids"][row:row + n].copy(),
                                   o["labels"][row:row + n].copy(), o["mask"][row:row + n].copy())
            row += n
    plan.destroy()
    pool.destroy()
    return res


@pytest.mark.parametrize("name,id_skew", [("image_mix_7b", "uniform"), ("video_heavy", "uniform"), ("image_mix_7b", "zipf")])
def test_full_size_backbone_side(name, id_skew):
    """Padded assembly and table gradient at the benchmark's size.  Rows: equal to the packed assembly (itself
    checked above), zero padding.  Ids, labels, mask: in full against the generator's ids.  Positions: sampled
    samples against the oracle.  Gradient: small-integer gradients against an exact scatter-add by a library
    routine, and sampled table rows of a real-valued run against sequential fp32 addition in row order."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import CudaRun, cuda_stream
    w = workloads.make_workload(name, id_skew=id_skew)   # zipf: a few ids own most text rows (the frequent-id path)
    run = CudaRun(w)
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        assert run.register(samples) == 0
        assert run.write(call, keep_src=False) == 0
    items = [(s, j, workloads.span_grid(w, s, j)) for s in range(w.n_samples) for j in range(int(w.n_spans[s]))]
    items = [it for it in items if it[2] is not None]
    assert run.pool.set_span_grids([s for s, _, _ in items], [j for _, j, _ in items], [g for _, _, g in items], cuda_stream()) == 0
    rc, plan = run.plan()
    assert rc == 0
    a = plan.arrays()
    n_mb, L, H = int(a["n_mb"]), w.budget_L, w.hidden
    rc, packed, _, packed_pos = run.gather_all()
    assert rc == 0
    lens = w.seq_len[a["mb_samples"]].astype(np.int64)
    all_ids = np.concatenate([workloads.input_ids(w, int(s)) for s in a["mb_samples"]])
    nxt_text = np.concatenate([np.append(workloads.input_ids(w, int(s))[1:] != w.placeholder_id, False) for s in a["mb_samples"]])
    nxt_id = np.concatenate([np.append(workloads.input_ids(w, int(s))[1:], 0) for s in a["mb_samples"]])
    picked = [int(s) for s in np.random.default_rng(3).choice(a["mb_samples"], size=5, replace=False)]
    exp_s = _oracle_samples(w, picked)
    per_call = max(1, min(n_mb, (1 << 20) // L))
    rows_cap = per_call * L
    out = torch.empty((rows_cap, H), dtype=torch.int16, device="cuda")
    cu = torch.empty((w.n_samples + 2 * n_mb,), dtype=torch.int32, device="cuda")
    pos3 = torch.empty((3 * rows_cap,), dtype=torch.int32, device="cuda")
    ids, labels = (torch.empty((rows_cap,), dtype=torch.int32, device="cuda") for _ in range(2))
    mask = torch.empty((rows_cap,), dtype=torch.uint8, device="cuda")
    row_off = np.concatenate([[0], np.cumsum(lens)])
    seen = 0
    for b in range(0, n_mb, per_call):
        e = min(n_mb, b + per_call)
        rows = (e - b) * L
        out.fill_(-1); pos3.fill_(-7); ids.fill_(-7); labels.fill_(-7); mask.fill_(7); cu.fill_(-7)
        assert run.pool.gather_padded(plan, b, e, run.table.data_ptr(), w.vocab, -2, out.data_ptr(), cu.data_ptr(), pos3.data_ptr(),
                                      ids.data_ptr(), labels.data_ptr(), mask.data_ptr(), cuda_stream()) == 0
        torch.cuda.synchronize()
        h_ids, h_lab, h_mask = ids[:rows].cpu().numpy(), labels[:rows].cpu().numpy(), mask[:rows].cpu().numpy()
        h_pos = pos3[:3 * rows].cpu().numpy().reshape(3, rows)
        h_cu = cu.cpu().numpy()
        cu_w = 0
        for j in range(b, e):
            q0, q1 = int(a["mb_sample_off"][j]), int(a["mb_sample_off"][j + 1])
            t = int(a["mb_tokens"][j])
            r0, R0 = int(row_off[q0]), (j - b) * L
            assert torch.equal(out[R0:R0 + t], packed[r0:r0 + t])
            assert not bool(out[R0 + t:R0 + L].any().item())
            assert np.array_equal(h_ids[R0:R0 + t], all_ids[r0:r0 + t]) and np.all(h_ids[R0 + t:R0 + L] == -2)
            assert np.array_equal(h_mask[R0:R0 + t], nxt_text[r0:r0 + t].astype(np.uint8)) and not h_mask[R0 + t:R0 + L].any()
            assert np.array_equal(h_lab[R0:R0 + t], np.where(nxt_text[r0:r0 + t], nxt_id[r0:r0 + t], -100)) and np.all(h_lab[R0 + t:R0 + L] == -100)
            assert not h_pos[:, R0 + t:R0 + L].any()
            exp_cu = np.concatenate([[0], np.cumsum(lens[q0:q1]), [L]]).astype(np.int32)
            assert np.array_equal(h_cu[cu_w:cu_w + len(exp_cu)], exp_cu)
            cu_w += len(exp_cu)
            for q in range(q0, q1):
                s = int(a["mb_samples"][q])
                if s in exp_s:
                    R = R0 + int(row_off[q]) - r0
                    n = int(lens[q])
                    assert np.array_equal(h_pos[:, R:R + n], exp_s[s][0]) and np.array_equal(h_lab[R:R + n], exp_s[s][2])
                    seen += 1
    assert seen == len(picked)
    del out
    # gradient, packed layout over the whole plan
    total = int(lens.sum())
    text_rows = torch.from_numpy(np.nonzero(all_ids != w.placeholder_id)[0]).cuda()
    text_ids = torch.from_numpy(all_ids[all_ids != w.placeholder_id].astype(np.int64)).cuda()
    grad = packed   # reuse the buffer: small integers first
    torch.manual_seed(5)
    step = 1 << 18
    for r in range(0, total, step):
        grad[r:r + step] = torch.randint(-8, 9, (min(step, total - r), H), device="cuda", dtype=torch.int16).to(torch.bfloat16).view(torch.int16)
    gt = torch.zeros((w.vocab, H), dtype=torch.float32, device="cuda")
    assert run.pool.embed_grad(plan, 0, n_mb, False, grad.data_ptr(), gt.data_ptr(), w.vocab, cuda_stream()) == 0
    ref = torch.zeros((w.vocab, H), dtype=torch.float32, device="cuda")
    for r in range(0, len(text_rows), step):
        ref.index_add_(0, text_ids[r:r + step], grad[text_rows[r:r + step]].view(torch.bfloat16).float())   # small integers: exact in any order
    torch.cuda.synchronize()
    assert torch.equal(gt, ref)
    del ref
    # real values: sampled table rows against sequential fp32 addition in ascending row order
    for r in range(0, total, step):
        grad[r:r + step] = workloads.grad_values(w, r, min(total, r + step), device="cuda").view(torch.int16)
    gt.zero_()
    assert run.pool.embed_grad(plan, 0, n_mb, False, grad.data_ptr(), gt.data_ptr(), w.vocab, cuda_stream()) == 0
    torch.cuda.synchronize()
    ids_np = all_ids
    counts = np.bincount(ids_np[ids_np != w.placeholder_id], minlength=w.vocab)
    for v in [int(np.argmax(counts)), int(np.argmin(np.where(counts > 0, counts, 1 << 30))), 17, w.vocab - 2]:
        rows_v = np.nonzero(ids_np == v)[0]
        acc = np.zeros(H, np.float32)
        g_rows = grad[torch.from_numpy(rows_v).cuda()].view(torch.bfloat16).float().cpu().numpy() if len(rows_v) else np.zeros((0, H), np.float32)
        for k in range(len(rows_v)):
            acc = acc + g_rows[k]          # float32 + float32, one rounding per element, in row order
        assert np.array_equal(gt[v].cpu().numpy().view(np.uint32), acc.view(np.uint32)), v
    assert run.pool.status() == (0, 0)
    run.close()


@pytest.mark.parametrize("page_bytes", [2 << 20, 4096])
def test_full_size_fragmentation_sweep(page_bytes):
    """Config 5 as bench.py runs it: a stream of 65 536 samples flows through a 64 GiB all-HBM pool (10 write/free
    cycles, final admit), then the residents are planned and assembled in ranges.  The plan is compared array by
    array with the oracle's Algorithm 1 on the residents' lengths; position ids and cu_seqlens in full with what the
    plan determines; sampled rows of every range with rows the generator gives one by one."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from gpu_harness import cuda_stream
    from harness import pool_config_fields, register_args, write_args
    from paper_2606_23087_b200 import binding as fp
    import gc
    gc.collect()
    torch.cuda.empty_cache()          # blocks cached by earlier tests of this process are not in use
    free_b, _ = torch.cuda.mem_get_info()
    pool_bytes = (64 << 30) if free_b >= (90 << 30) else (32 << 30)
    w = workloads.make_workload("frag_sweep", n_samples=65536, page_bytes=page_bytes, pool_bytes=pool_bytes)
    ops, residents = workloads.admit_free_schedule(w, cycles=10)
    pool = fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    st = cuda_stream()
    for kind, samples in ops:
        if kind == "free":
            assert pool.free(samples, st) == 0
            continue
        for i in range(0, len(samples), 256):
            part = samples[i:i + 256]
            reg = register_args(w, part)
            ids = torch.from_numpy(reg[5]).cuda()
            srcs = [workloads.span_values(w, s, 0, device="cuda") for s in part]
            assert pool.register_samples(*reg[:5], ids.data_ptr(), st) == 0
            assert pool.write_embeddings(*write_args(w, [(s, 0) for s in part]), [t.data_ptr() for t in srcs], 0, st) == 0
            torch.cuda.synchronize()
    assert pool.status() == (0, 0)
    order = np.asarray(residents, dtype=np.uint32)
    cfg = plan_config_fields(w)
    rc, plan = pool.plan_microbatches(order, fp.PlanConfig(**cfg), st)
    assert rc == 0
    got = plan.arrays()
    rc, oplan = plan_from_lengths(w.seq_len[order], PlanConfig(**cfg), slots=order)
    assert rc == 0
    exp = oplan.arrays()
    for k in PLAN_KEYS:
        assert np.array_equal(got[k], exp[k]), k
    n_mb, total, _ = plan.summary()
    assert (n_mb, total) == oplan.summary()[:2] and len(residents) > (8000 if pool_bytes == (64 << 30) else 4000)
    table = workloads.embed_table(w, device="cuda")
    buf_rows = min(total, 1 << 20)
    out = torch.empty((buf_rows, w.hidden), dtype=torch.int16, device="cuda")
    cu = torch.empty((len(residents) + n_mb + 8,), dtype=torch.int32, device="cuda")
    pos = torch.empty((buf_rows,), dtype=torch.int32, device="cuda")
    lens = w.seq_len[exp["mb_samples"]].astype(np.int64)
    row_off = np.concatenate([[0], np.cumsum(lens)])
    mb_row = np.concatenate([[0], np.cumsum(exp["mb_tokens"].astype(np.int64))])
    ranges, b, rows = [], 0, 0
    for j in range(n_mb):
        t = int(exp["mb_tokens"][j])
        if rows + t > buf_rows:
            ranges.append((b, j)); b, rows = j, 0
        rows += t
    ranges.append((b, n_mb))
    rng = np.random.default_rng(17)
    table_i16 = table.view(torch.int16)
    covered = 0
    for lo, hi in ranges:
        out.fill_(-1)
        assert pool.gather_packed(plan, lo, hi, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), st) == 0
        torch.cuda.synchronize()
        q0, q1 = int(exp["mb_sample_off"][lo]), int(exp["mb_sample_off"][hi])
        n_rows = int(mb_row[hi] - mb_row[lo])
        exp_pos = np.concatenate([np.arange(l, dtype=np.int32) for l in lens[q0:q1]])
        assert np.array_equal(pos[:n_rows].cpu().numpy(), exp_pos)
        exp_cu = np.concatenate([np.concatenate([[0], np.cumsum(lens[int(exp["mb_sample_off"][j]):int(exp["mb_sample_off"][j + 1])])])
                                 for j in range(lo, hi)]).astype(np.int32)
        assert np.array_equal(cu[:len(exp_cu)].cpu().numpy(), exp_cu)
        assert not bool((out[:n_rows] == -1).all(dim=1).any().item())
        # every row of the range against the generator
        covered += assert_every_row(w, out, exp["mb_samples"][q0:q1], row_off[q0:q1] - mb_row[lo], table_i16)
        picks = []
        for q in rng.choice(np.arange(q0, q1), size=min(6, q1 - q0), replace=False):
            s = int(exp["mb_samples"][q])
            sp, tk = w.spans_of(s)
            for p in {0, int(lens[q]) - 1, int(sp[0]), int(sp[0]) + int(tk[0]) - 1, int(rng.integers(0, lens[q]))}:
                picks.append((int(row_off[q] - mb_row[lo]) + p, s, p))
        got_rows = out[torch.tensor([r for r, _, _ in picks], device="cuda")].cpu().numpy().view(np.uint16)
        for i, (_, s, p) in enumerate(picks):
            assert np.array_equal(got_rows[i], expected_row(w, s, p)), (lo, hi, s, p)
    assert covered == len(residents)
    assert pool.status() == (0, 0)
    plan.destroy(); oplan.destroy()
    pool.destroy()
