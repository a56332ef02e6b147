"""pool_write_embeddings_noalloc against pool_write_embeddings, through the C ABI, on a GPU.

Some callers of the write path may not allocate device or pinned memory at the moment they call it (a
producer inside a region where the framework's allocator is frozen, a loop that cannot take cudaMalloc's
implicit synchronisation).  The no-alloc entry point keeps its per-call scratch in a fixed device array
instead.  This test writes the same embeddings through both entry points into two pools of identical
configuration, on two producer calls in a row (the second call finds the first call's descriptors still in
the shared array), and requires identical page lists and bit-identical assembled output -- the same
bit-exact bar as every other GPU test here -- and the same again against the CPU oracle.  A second case fills
the fixed array to its limit: 4096 one-token spans in one call on an all-HBM pool with 4 KiB pages.  The file
name sorts last so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

import workloads
from harness import plan_config_fields, pool_config_fields, register_args, run_oracle, write_args

pytestmark = pytest.mark.gpu


def _run(w, use_noalloc):
    from gpu_harness import cuda_stream
    from paper_2606_23087_b200 import binding as fp
    pool = fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    keep = []
    for call in w.write_calls:                       # two calls in a row
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        a = register_args(w, samples)
        ids = torch.from_numpy(a[5]).cuda()
        srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]
        keep += [ids, srcs]
        assert pool.register_samples(*a[:5], ids.data_ptr(), cuda_stream()) == 0
        write = pool.write_embeddings_noalloc if use_noalloc else pool.write_embeddings
        assert write(*write_args(w, call), [t.data_ptr() for t in srcs], w.src_dtype, cuda_stream()) == 0
    pages = {(s, j): pool.span_pages(s, j)[1] for call in w.write_calls for s, j in call}
    rc, plan = pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), fp.PlanConfig(**plan_config_fields(w)),
                                      cuda_stream())
    assert rc == 0
    n_mb, total, _ = plan.summary()
    table = workloads.embed_table(w, device="cuda")
    out = torch.full((total, w.hidden), -1, dtype=torch.int16, device="cuda")
    cu = torch.full((w.n_samples + n_mb,), -1, dtype=torch.int32, device="cuda")
    pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
    assert pool.gather_packed(plan, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(),
                              cuda_stream()) == 0
    torch.cuda.synchronize()
    status = pool.status()
    res = (pages, out.cpu().numpy(), cu.cpu().numpy(), pos.cpu().numpy(), status, pool.stats()["pages_free"])
    plan.destroy()
    pool.destroy()
    return res


@pytest.mark.parametrize("name,kw", [
    ("image_mix_7b", dict(n_samples=12, hidden=512, page_bytes=65536)),      # two tiers, bf16 source
    ("host_tier_stress", dict(n_samples=4, hidden=256, page_bytes=65536)),   # fp32 source with the fused cast
])
def test_noalloc_write_matches_regular_write(name, kw):
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    w = workloads.make_workload(name, **kw)
    half = w.n_samples // 2
    order = list(range(w.n_samples))
    w.write_calls = [[(s, j) for s in part for j in range(int(w.n_spans[s]))] for part in (order[:half], order[half:])]
    w.plan_order = order
    ref = _run(w, use_noalloc=False)
    got = _run(w, use_noalloc=True)
    assert got[0].keys() == ref[0].keys()
    for k in ref[0]:
        assert np.array_equal(got[0][k], ref[0][k]), k
    for a, b in zip(got[1:4], ref[1:4]):
        assert np.array_equal(a, b)                  # bit-exact, as everywhere in this suite
    assert got[4] == ref[4] == (0, 0) and got[5] == ref[5]
    assert not np.any(np.all(got[1] == -1, axis=1))
    _assert_equals_oracle(w, got)


def _assert_equals_oracle(w, got):
    """The same call sequence through the CPU oracle: page lists, rows, cu_seqlens, position ids."""
    exp = run_oracle(w)
    assert all(rc == 0 for rc in exp["rc"]) and exp["status"] == (0, 0)
    for k, pages in exp["span_pages"].items():
        assert np.array_equal(got[0][k], pages), k
    assert np.array_equal(got[1].view(np.uint16), exp["out"])
    assert np.array_equal(got[2], exp["cu_seqlens"]) and np.array_equal(got[3], exp["position_ids"])


def test_noalloc_at_its_span_limit_on_an_all_hbm_pool():
    """FT_NOALLOC_MAX_SPANS spans in ONE call: the fixed array is used up to its last descriptor slot, the copy
    kernel finds each chunk's span by search (the array has no room for a per-chunk table), and with every page in
    HBM the whole call is one launch.  1024 samples x 4 one-token spans, hidden 64, 4 KiB pages (one page per span)."""
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2606_23087_b200 import binding as fp
    from workloads.gen import _assemble
    n = fp.FT_NOALLOC_MAX_SPANS // 4
    w = _assemble("span_limit", 7, 64, 4096, np.full(n, 8), [[1, 1, 1, 1]] * n, budget_L=4096)
    w.hbm_pages, w.host_pages = 4 * n + 16, 0
    order = list(range(n))
    w.write_calls = [[(s, j) for s in order for j in range(4)]]
    w.plan_order = order
    assert len(w.write_calls[0]) == fp.FT_NOALLOC_MAX_SPANS
    ref = _run(w, use_noalloc=False)
    got = _run(w, use_noalloc=True)
    for k in ref[0]:
        assert np.array_equal(got[0][k], ref[0][k]), k
    for a, b in zip(got[1:4], ref[1:4]):
        assert np.array_equal(a, b)
    assert got[4] == ref[4] == (0, 0) and got[5] == ref[5] == 16
    _assert_equals_oracle(w, got)


def test_noalloc_rejects_oversized_calls():
    if not torch.cuda.is_available():
        pytest.fail("a CUDA device is required for -m gpu tests")
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload("tiny", hidden=64, page_bytes=4096)
    pool = fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
    n = fp.FT_NOALLOC_MAX_SPANS + 1
    z = np.zeros(n, np.uint32)
    assert pool.write_embeddings_noalloc(z, z, z, np.ones(n, np.uint64), 0) == -11   # FT_ERR_CAPACITY, nothing done
    assert pool.stats()["pages_free"] == w.hbm_pages
    pool.destroy()
