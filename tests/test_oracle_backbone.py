"""Pins for the oracle's backbone-side outputs (padded layout, three-component positions, labels and loss
mask, table gradient): hand-worked fixtures, reductions to the packed assembly, and library routines on cases
where the order of additions cannot matter.  CPU only."""
import os

import numpy as np
import torch

import workloads
from harness import bits16, pool_config_fields, plan_config_fields, register_args, run_oracle, write_args, host_span
from oracle import OraclePool, PlanConfig, PoolConfig
from test_oracle_pins import golden, plan_cfg, small_pool


def hand_sample(grids):
    """The fixture's 19-position sample in a small pool, written and planned alone (L = 24)."""
    g = golden("backbone_hand.txt")
    pool = small_pool(hidden=8, hbm_pages=4, host_pages=0)
    ids = np.array(g["P_ids"], np.int32)
    assert pool.register_samples([0], [g["P_seq_len"][0]], [2], g["P_span_pos"], g["P_span_tokens"], ids) == 0
    rng = np.random.default_rng(0)
    srcs = [rng.integers(0, 0x7F00, size=(n, 8)).astype(np.uint16) for n in g["P_span_tokens"]]
    assert pool.write_embeddings([0, 0], [0, 1], g["P_span_tokens"], srcs, 0) == 0
    if grids:
        assert pool.set_span_grids([0] * len(grids), list(grids.keys()), list(grids.values())) == 0
    rc, plan = pool.plan_microbatches([0], plan_cfg(g["P_L"][0]))
    assert rc == 0
    return g, pool, plan, srcs


def padded_outputs(pool, plan, n_mb, L, H, table, pad_id):
    rows = n_mb * L
    o = dict(out=np.full((rows, H), 0xFFFF, np.uint16), cu=np.full(plan.n + 2 * n_mb, -7, np.int32),
             pos3=np.full((3, rows), -7, np.int32), ids=np.full(rows, -7, np.int32), labels=np.full(rows, -7, np.int32),
             mask=np.full(rows, 7, np.uint8))
    rc = pool.gather_padded(plan, 0, n_mb, table, pad_id, o["out"], o["cu"], o["pos3"], o["ids"], o["labels"], o["mask"])
    assert rc == 0, rc
    return o


def test_hand_example_positions_labels_padding():
    g, pool, plan, srcs = hand_sample({0: g_a(), 1: g_b()})
    table = np.arange(100 * 8, dtype=np.uint16).reshape(100, 8)
    L, n = g["P_L"][0], g["P_seq_len"][0]
    o = padded_outputs(pool, plan, 1, L, 8, table, g["P_pad_id"][0])
    assert list(o["pos3"][0, :n]) == g["P_pos_t"] and list(o["pos3"][1, :n]) == g["P_pos_h"] and list(o["pos3"][2, :n]) == g["P_pos_w"]
    assert list(o["ids"][:n]) == g["P_ids"] and list(o["labels"][:n]) == g["P_labels"] and list(o["mask"][:n]) == g["P_mask"]
    assert list(o["cu"]) == g["P_cu"]
    assert np.all(o["pos3"][:, n:] == 0) and np.all(o["ids"][n:] == g["P_pad_id"][0])
    assert np.all(o["labels"][n:] == -100) and np.all(o["mask"][n:] == 0) and np.all(o["out"][n:] == 0)
    # rows: text rows are table rows, span rows are the written images
    assert np.array_equal(o["out"][0], table[5]) and np.array_equal(o["out"][8], table[7]) and np.array_equal(o["out"][18], table[9])
    assert np.array_equal(o["out"][2:8], srcs[0]) and np.array_equal(o["out"][10:18], srcs[1])
    assert pool.status() == (0, 0)


def g_a():
    return golden("backbone_hand.txt")["P_grid_A"]


def g_b():
    return golden("backbone_hand.txt")["P_grid_B"]


def test_span_without_grid_counts_as_text():
    g, pool, plan, _ = hand_sample({0: g_a()})
    table = np.zeros((100, 8), np.uint16)
    n = g["P_seq_len"][0]
    o = padded_outputs(pool, plan, 1, g["P_L"][0], 8, table, -1)
    for c, k in enumerate(("P_nogridB_pos_t", "P_nogridB_pos_h", "P_nogridB_pos_w")):
        assert list(o["pos3"][c, :n]) == g[k]


def test_grid_argument_checks_are_all_or_nothing():
    g, pool, plan, _ = hand_sample(None)
    assert pool.set_span_grids([0], [0], [[1, 2, 4]]) == -1          # 8 tokens != 6
    assert pool.set_span_grids([0], [0], [[0, 2, 3]]) == -1          # zero extent
    assert pool.set_span_grids([0], [2], [[1, 2, 3]]) == -1          # no such span
    assert pool.set_span_grids([1], [0], [[1, 2, 3]]) == -3          # slot not registered
    assert pool.set_span_grids([9], [0], [[1, 2, 3]]) == -1          # slot out of range
    assert pool.set_span_grids([0, 0], [0, 1], [[1, 2, 3], [3, 3, 1]]) == -1   # second item bad: first not stored
    table = np.zeros((100, 8), np.uint16)
    o = padded_outputs(pool, plan, 1, g["P_L"][0], 8, table, -1)
    n = g["P_seq_len"][0]
    assert all(list(o["pos3"][c, :n]) == list(range(n)) for c in range(3))   # no grid anywhere: plain positions


def build_tiny(n_samples=16, with_grids=True):
    w = workloads.make_workload("tiny", n_samples=n_samples)
    res = run_oracle(w, keep_pool=True)
    pool, plan = res["pool"], res["plan_handle"]
    if with_grids:
        items = [(s, j, workloads.span_grid(w, s, j)) for s in range(w.n_samples) for j in range(int(w.n_spans[s]))]
        items = [it for it in items if it[2] is not None]
        assert pool.set_span_grids([s for s, _, _ in items], [j for _, j, _ in items], [gr for _, _, gr in items]) == 0
    return w, res, pool, plan


def test_padded_layout_reduces_to_the_packed_assembly():
    w, res, pool, plan = build_tiny(with_grids=False)
    a, L, H = res["plan"], w.budget_L, w.hidden
    n_mb = a["n_mb"]
    o = padded_outputs(pool, plan, n_mb, L, H, res["table"], w.placeholder_id)
    row = cu_r = cu_w = 0
    for j in range(n_mb):
        t = int(a["mb_tokens"][j])
        nj = int(a["mb_sample_off"][j + 1] - a["mb_sample_off"][j])
        assert np.array_equal(o["out"][j * L:j * L + t], res["out"][row:row + t])
        assert np.all(o["out"][j * L + t:(j + 1) * L] == 0)
        # without grids all three components are the packed position ids
        for c in range(3):
            assert np.array_equal(o["pos3"][c, j * L:j * L + t], res["position_ids"][row:row + t])
        assert list(o["cu"][cu_w:cu_w + nj + 1]) == list(res["cu_seqlens"][cu_r:cu_r + nj + 1]) and o["cu"][cu_w + nj + 1] == L
        row += t; cu_r += nj + 1; cu_w += nj + 2
    assert pool.status() == (0, 0)


def test_ids_and_labels_follow_the_generator_inputs():
    w, res, pool, plan = build_tiny()
    a, L = res["plan"], w.budget_L
    o = padded_outputs(pool, plan, a["n_mb"], L, w.hidden, res["table"], -5)
    for j in range(a["n_mb"]):
        row = j * L
        for s in a["mb_samples"][a["mb_sample_off"][j]:a["mb_sample_off"][j + 1]]:
            ids = workloads.input_ids(w, int(s))
            n = len(ids)
            assert np.array_equal(o["ids"][row:row + n], ids)
            nxt_is_text = np.append(ids[1:] != w.placeholder_id, False)   # generator ids never equal the placeholder off-span
            exp = np.where(nxt_is_text, np.append(ids[1:], 0), -100)
            assert np.array_equal(o["labels"][row:row + n], exp)
            assert np.array_equal(o["mask"][row:row + n], nxt_is_text.astype(np.uint8))
            row += n
        assert np.all(o["ids"][row:(j + 1) * L] == -5) and np.all(o["labels"][row:(j + 1) * L] == -100)


def test_positions_with_grids_properties():
    """Per sample: a text token's three components are equal; after a span the counter continues at the span's
    start + its largest extent; inside a span the components enumerate the grid row-major."""
    w, res, pool, plan = build_tiny()
    a, L = res["plan"], w.budget_L
    o = padded_outputs(pool, plan, a["n_mb"], L, w.hidden, res["table"], 0)
    seen_grid = 0
    for j in range(a["n_mb"]):
        row = j * L
        for s in a["mb_samples"][a["mb_sample_off"][j]:a["mb_sample_off"][j + 1]]:
            s = int(s)
            n = int(w.seq_len[s])
            p3 = o["pos3"][:, row:row + n]
            pos, tok = w.spans_of(s)
            st, p = 0, 0
            for k in range(len(pos)):
                while p < int(pos[k]):
                    assert tuple(p3[:, p]) == (st, st, st); st += 1; p += 1
                gr = workloads.span_grid(w, s, k)
                if gr is None:
                    for _ in range(int(tok[k])):
                        assert tuple(p3[:, p]) == (st, st, st); st += 1; p += 1
                else:
                    seen_grid += 1
                    T, H, W = gr
                    block = p3[:, p:p + T * H * W].reshape(3, T, H, W) - st
                    tt, hh, ww = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
                    assert np.array_equal(block[0], tt) and np.array_equal(block[1], hh) and np.array_equal(block[2], ww)
                    st += max(gr); p += T * H * W
            while p < n:
                assert tuple(p3[:, p]) == (st, st, st); st += 1; p += 1
            row += n
    assert seen_grid >= 8


def test_table_gradient_hand_order():
    g = golden("backbone_hand.txt")
    for vals, want in ((g["G_values_a"], g["G_sum_a"][0]), (g["G_values_b"], g["G_sum_b"][0])):
        pool = small_pool(hidden=8, hbm_pages=2, host_pages=0)
        assert pool.register_samples([0], [3], [0], [], [], np.array([4, 4, 4], np.int32)) == 0
        rc, plan = pool.plan_microbatches([0], plan_cfg(8))
        grad = np.zeros((3, 8), np.uint16)
        grad[:, 0] = bits16(torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16))
        grad[:, 1] = bits16(torch.tensor([1.5, -0.25, 2.0]).to(torch.bfloat16))
        table = np.zeros((10, 8), np.float32)
        table[4, 2] = 3.0   # accumulates onto what is there
        assert pool.embed_grad(plan, 0, 1, False, grad, table) == 0
        assert table[4, 0] == np.float32(want) and table[4, 1] == np.float32(3.25) and table[4, 2] == 3.0
        assert np.count_nonzero(table) == 3


def test_table_gradient_integer_case_matches_add_at():
    """Small-integer gradients: every partial sum is exact in fp32, so any order gives the same table and
    numpy's unordered scatter-add is the definition."""
    w, res, pool, plan = build_tiny()
    a, L, H = res["plan"], w.budget_L, w.hidden
    n_mb = a["n_mb"]
    rng = np.random.default_rng(5)
    for padded in (False, True):
        rows = n_mb * L if padded else int(a["mb_tokens"].sum())
        gi = rng.integers(-64, 65, size=(rows, H))
        grad = bits16(torch.from_numpy(gi.astype(np.float32)).to(torch.bfloat16))
        table = np.zeros((w.vocab, H), np.float32)
        assert pool.embed_grad(plan, 0, n_mb, padded, grad, table) == 0
        exp = np.zeros((w.vocab, H), np.int64)
        row0 = 0
        for j in range(n_mb):
            row = j * L if padded else row0
            for s in a["mb_samples"][a["mb_sample_off"][j]:a["mb_sample_off"][j + 1]]:
                ids = workloads.input_ids(w, int(s))
                text = ids != w.placeholder_id
                np.add.at(exp, ids[text], gi[row:row + len(ids)][text])
                row += len(ids)
            row0 += int(a["mb_tokens"][j])
        assert np.array_equal(table.astype(np.int64), exp) and np.array_equal(table, exp.astype(np.float32))
    # a sub-range touches only its own rows: two half-range calls accumulate to the full-range result
    rows = int(a["mb_tokens"].sum())
    grad = bits16(workloads.grad_values(w, 0, rows))
    full = np.zeros((w.vocab, H), np.float32)
    assert pool.embed_grad(plan, 0, n_mb, False, grad, full) == 0
    if n_mb >= 2:
        t0 = int(a["mb_tokens"][0])
        two = np.zeros((w.vocab, H), np.float32)
        assert pool.embed_grad(plan, 0, 1, False, grad[:t0], two) == 0
        assert pool.embed_grad(plan, 1, n_mb, False, grad[t0:], two) == 0
        assert np.array_equal(two.view(np.uint32), full.view(np.uint32))
    # and the general case agrees with a float64 scatter-add to rounding
    exp = np.zeros((w.vocab, H), np.float64)
    row = 0
    gv = workloads.grad_values(w, 0, rows).to(torch.float64).numpy()
    for j in range(n_mb):
        for s in a["mb_samples"][a["mb_sample_off"][j]:a["mb_sample_off"][j + 1]]:
            ids = workloads.input_ids(w, int(s))
            text = ids != w.placeholder_id
            np.add.at(exp, ids[text], gv[row:row + len(ids)][text])
            row += len(ids)
    assert np.allclose(full, exp, rtol=1e-5, atol=1e-5)


def test_list_assembly_is_the_concatenation_of_single_microbatch_assemblies():
    """A rank consumes the microbatches dealt to it (Algorithm 1, lines 15-27), not a contiguous range."""
    w = workloads.make_workload("image_mix_7b", n_samples=40, hidden=56, page_bytes=4096)
    w.budget_L = int(w.seq_len.max())   # several microbatches
    res = run_oracle(w, keep_pool=True)
    pool, plan, a = res["pool"], res["plan_handle"], res["plan"]
    n_mb, H = int(a["n_mb"]), w.hidden
    assert n_mb >= 6
    tok = a["mb_tokens"].astype(np.int64)
    row_off = np.concatenate([[0], np.cumsum(tok)])
    cu_off = np.concatenate([[0], np.cumsum(np.diff(a["mb_sample_off"].astype(np.int64)) + 1)])

    def by_list(lst):
        rows = int(tok[lst].sum()) if len(lst) else 0
        n_cu = int(sum(cu_off[j + 1] - cu_off[j] for j in lst))
        out = np.full((max(rows, 1), H), 0xFFFF, np.uint16)
        cu = np.full(max(n_cu, 1), -7, np.int32)
        pos = np.full(max(rows, 1), -7, np.int32)
        assert pool.gather_list(plan, lst, res["table"], out, cu, pos) == 0
        return out[:rows], cu[:n_cu], pos[:rows]

    # the identity list is the full-range assembly
    out, cu, pos = by_list(list(range(n_mb)))
    assert np.array_equal(out, res["out"]) and np.array_equal(cu, res["cu_seqlens"]) and np.array_equal(pos, res["position_ids"])
    # every rank's list, a reversed list and a list with a repeat: slices of the full-range assembly, in list order
    lists = [list(a["rank_mbs"][a["rank_mb_off"][r]:a["rank_mb_off"][r + 1]]) for r in range(w.n_ranks_N)]
    lists += [list(range(n_mb))[::-1], [2, 2, 0]]
    assert sorted(j for l in lists[:w.n_ranks_N] for j in l) == list(range(n_mb))
    for lst in lists:
        lst = [int(j) for j in lst]
        out, cu, pos = by_list(lst)
        exp_out = np.concatenate([res["out"][row_off[j]:row_off[j + 1]] for j in lst]) if lst else np.zeros((0, H), np.uint16)
        exp_cu = np.concatenate([res["cu_seqlens"][cu_off[j]:cu_off[j + 1]] for j in lst]) if lst else np.zeros(0, np.int32)
        exp_pos = np.concatenate([res["position_ids"][row_off[j]:row_off[j + 1]] for j in lst]) if lst else np.zeros(0, np.int32)
        assert np.array_equal(out, exp_out) and np.array_equal(cu, exp_cu) and np.array_equal(pos, exp_pos)
    one = np.zeros((1, H), np.uint16); c1 = np.zeros(1, np.int32)
    assert pool.gather_list(plan, [n_mb], res["table"], one, c1, c1) == -1      # no such microbatch
    assert pool.gather_list(plan, [], res["table"], one, c1, c1) == 0
    # an id outside the table: reported with the row index in the list's output
    small = res["table"][:100]
    lst = [3, 1]
    rows = int(tok[lst].sum())
    out = np.full((rows, H), 0xFFFF, np.uint16); cu = np.zeros(64, np.int32); pos = np.zeros(rows, np.int32)
    assert pool.gather_list(plan, lst, small, out, cu, pos) == 0
    code, detail = pool.status()
    ids3 = np.concatenate([workloads.input_ids(w, int(s)) for s in a["mb_samples"][a["mb_sample_off"][3]:a["mb_sample_off"][4]]])
    first_bad = int(np.nonzero((ids3 != w.placeholder_id) & (ids3 >= 100))[0][0])
    assert (code, detail) == (-9, first_bad)
    assert pool.free([int(a["mb_samples"][0])]) == 0
    assert pool.gather_list(plan, [0], res["table"], out, cu, pos) == -5        # the plan died with its sample
    plan.destroy(); pool.destroy()
