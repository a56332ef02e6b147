"""The seeded input generator: shapes and ranges of the five configurations, determinism, and the prefix property
(a smaller case is the beginning of the full one).  CPU only."""
import numpy as np
import torch

import workloads


def test_config_shapes_and_ranges():
    w = workloads.make_workload("tiny")
    assert w.n_samples == 16 and w.hidden == 1024 and w.page_bytes == 64 << 10 and w.budget_L == 4096
    assert np.all(w.n_spans == 1) and np.all((w.span_tokens >= 64) & (w.span_tokens <= 256)) and w.host_pages == 0
    w = workloads.make_workload("image_mix_7b")
    assert w.n_samples == 512 and w.hidden == 3584 and w.page_bytes == 2 << 20 and w.budget_L == 32768
    assert np.all((w.n_spans >= 1) & (w.n_spans <= 4)) and np.all((w.span_tokens >= 256) & (w.span_tokens <= 4096))
    text = w.seq_len.astype(np.int64) - np.array([w.spans_of(s)[1].sum() for s in range(512)])
    assert text.min() >= 128 and text.max() <= 4096
    P = w.hbm_pages + w.host_pages
    assert abs(w.hbm_pages / P - 0.8) < 0.001 and len(w.write_calls) == 16 and w.coef_A == 12 * 3584
    assert 900 < np.median(w.span_tokens) < 1150          # log-normal with median 1024
    w = workloads.make_workload("video_heavy")
    assert w.n_samples == 128 and np.all(w.span_tokens == 256) and np.all((w.n_spans >= 8) & (w.n_spans <= 64))
    assert sorted(w.plan_order) == list(range(128)) and w.plan_order != list(range(128))   # random completion order
    assert w.pages_of_span(256) == 1 and w.host_pages == 0 and w.budget_L == 131072
    w = workloads.make_workload("host_tier_stress")
    assert w.n_samples == 256 and w.hidden == 8192 and w.src_dtype == 1 and w.ring_order == 1
    assert w.hbm_pages == w.host_pages and np.all((w.span_tokens >= 2048) & (w.span_tokens <= 8192))
    w = workloads.make_workload("frag_sweep", n_samples=4096, pool_bytes=1 << 30, page_bytes=4096)
    assert np.all((w.span_tokens >= 64) & (w.span_tokens <= 16384)) and w.hbm_pages == (1 << 30) // 4096


def test_runs_are_sorted_and_inside_the_sequence():
    for name in ("image_mix_7b", "video_heavy"):
        w = workloads.make_workload(name, n_samples=40)
        for s in range(w.n_samples):
            pos, tok = w.spans_of(s)
            ends = pos.astype(np.int64) + tok
            assert np.all(pos[1:] >= ends[:-1]) and ends[-1] <= w.seq_len[s]
            ids = workloads.input_ids(w, s)
            mask = np.zeros(len(ids), bool)
            for p, t in zip(pos, tok):
                mask[int(p):int(p) + int(t)] = True
            assert np.array_equal(ids == w.placeholder_id, mask) and ids[~mask].max(initial=0) <= w.vocab - 2


def test_generator_is_deterministic_and_prefix_stable():
    a = workloads.make_workload("image_mix_7b", n_samples=24)
    b = workloads.make_workload("image_mix_7b", n_samples=512)
    assert np.array_equal(a.seq_len, b.seq_len[:24]) and np.array_equal(a.span_tokens, b.span_tokens[:len(a.span_tokens)])
    assert np.array_equal(workloads.input_ids(a, 5), workloads.input_ids(b, 5))
    x, y = workloads.span_values(a, 3, 0), workloads.span_values(b, 3, 0)
    assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    part = workloads.span_values(a, 3, 0, rows=(10, 14))
    assert torch.equal(part.view(torch.int16), x[10:14].view(torch.int16))      # a row range is a slice of the whole
    t = workloads.embed_table(a, rows=(7, 9))
    assert torch.equal(t.view(torch.int16), workloads.embed_table(b, rows=(0, 16))[7:9].view(torch.int16))


def test_values_look_like_unit_normal_and_specials_are_injected():
    w = workloads.make_workload("tiny")
    x = torch.cat([workloads.span_values(w, s, 0) for s in range(4)]).float()
    assert abs(x.mean().item()) < 0.01 and abs(x.std().item() - 1.0) < 0.01 and x.abs().max().item() < 3.5
    w4 = workloads.make_workload("host_tier_stress", n_samples=2, hidden=64)
    v = workloads.span_values(w4, 0, 0).view(torch.int32).flatten().numpy().view(np.uint32)
    spec = workloads.special_f32_bits()
    hits = v[::4099]
    assert np.array_equal(hits[:len(spec)], spec)          # every 4099th element cycles through the special patterns
    assert np.isnan(v.view(np.float32)).sum() > 0


def test_churn_schedule_respects_capacity():
    w = workloads.make_workload("frag_sweep", n_samples=3000, pool_bytes=256 << 20, page_bytes=65536, hidden=1024)
    ops, residents = workloads.admit_free_schedule(w, cycles=5)
    free = w.hbm_pages
    live = []
    for kind, samples in ops:
        need = sum(w.pages_of_span(int(w.spans_of(s)[1][0])) for s in samples)
        if kind == "admit":
            assert need <= free
            free -= need
            live += samples
        else:
            assert set(samples) <= set(live)
            free += need
            live = [s for s in live if s not in set(samples)]
    assert live == residents and sorted(live) == live        # admission order
    nxt = max(live) + 1
    assert nxt >= w.n_samples or w.pages_of_span(int(w.spans_of(nxt)[1][0])) > free   # the pool is full


def test_zipf_like_ids_and_span_grids():
    w = workloads.make_workload("image_mix_7b", n_samples=24, id_skew="zipf")
    u = workloads.make_workload("image_mix_7b", n_samples=24)
    ids = np.concatenate([workloads.input_ids(w, s) for s in range(w.n_samples)])
    text = ids[ids != w.placeholder_id]
    assert text.min() >= 0 and text.max() <= w.vocab - 2
    # log-uniform: id 0 holds ln 2 / ln(vocab - 1) of the text tokens, and the layout is the uniform workload's
    share0 = float((text == 0).mean())
    assert abs(share0 - np.log(2.0) / np.log(w.vocab - 1.0)) < 0.01
    assert np.array_equal(w.seq_len, u.seq_len) and np.array_equal(w.span_pos, u.span_pos)
    assert np.array_equal(workloads.input_ids(w, 3), workloads.input_ids(w, 3))
    for s in range(w.n_samples):
        pos, tok = w.spans_of(s)
        row = workloads.input_ids(w, s)
        for j in range(len(pos)):
            assert np.all(row[int(pos[j]):int(pos[j]) + int(tok[j])] == w.placeholder_id)
            g = workloads.span_grid(w, s, j)
            if g is not None:
                assert g[0] * g[1] * g[2] == int(tok[j]) and min(g) >= 1 and g[0] in (1, 2) and g[2] <= g[1]
    grids = [workloads.span_grid(w, s, j) for s in range(w.n_samples) for j in range(int(w.n_spans[s]))]
    assert any(g is None for g in grids) and any(g is not None and g[0] == 2 for g in grids)
    g0 = workloads.grad_values(w, 5, 9)
    assert g0.dtype == torch.bfloat16 and g0.shape == (4, w.hidden) and torch.equal(g0, workloads.grad_values(w, 5, 9))
    assert torch.equal(g0[1:], workloads.grad_values(w, 6, 9))   # a pure function of the row index
