"""Drives one implementation of the pool calls over a synthetic workload.

`run_oracle` feeds the CPU oracle; the GPU tests have a twin in
test_gpu_parity.py that feeds the CUDA library the same argument sequence.
Nothing here computes anything the method computes: it only builds arguments
from a workloads.Workload and collects outputs.
"""
import numpy as np
import torch

import workloads
from oracle import OraclePool, PlanConfig, PoolConfig


def bits16(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bits32(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int32).cpu().numpy().view(np.uint32)


def pool_config_fields(w, max_samples=None, ring_seed=11, bind_seed=12):
    return dict(
        page_bytes=w.page_bytes, hbm_pages=w.hbm_pages, host_pages=w.host_pages,
        max_text_tokens=w.total_text_tokens_capacity, ring_seed=ring_seed, bind_seed=bind_seed,
        gva_hbm_start=0, gva_host_start=0, max_size=0, hidden=w.hidden,
        max_samples=max_samples or w.n_samples, max_spans_per_sample=w.max_spans_per_sample,
        max_pages_per_span=w.max_pages_per_span, max_seq_len=w.max_seq_len,
        placeholder_id=w.placeholder_id, ring_order=w.ring_order, bind_order=w.bind_order,
        world_size=1, rank=0, max_imported_pages=0,
    )


def plan_config_fields(w, flags=0):
    return dict(coef_A=w.coef_A, coef_B=w.coef_B, budget_L=w.budget_L, n_buckets_K=w.n_buckets_K,
                n_ranks_N=w.n_ranks_N, flags=flags)


def register_args(w, samples):
    """Argument arrays of one pool_register_samples call for the given sample ids (slot = sample id)."""
    slots = np.asarray(samples, dtype=np.uint32)
    seq_len = w.seq_len[samples].astype(np.uint32)
    n_spans = w.n_spans[samples].astype(np.uint32)
    pos = np.concatenate([w.spans_of(s)[0] for s in samples]) if len(samples) else np.zeros(0, np.uint32)
    tok = np.concatenate([w.spans_of(s)[1] for s in samples]) if len(samples) else np.zeros(0, np.uint32)
    ids = np.concatenate([workloads.input_ids(w, s) for s in samples]) if len(samples) else np.zeros(0, np.int32)
    return slots, seq_len, n_spans, pos.astype(np.uint32), tok.astype(np.uint32), ids.astype(np.int32)


def write_args(w, call):
    slots = np.array([s for s, _ in call], dtype=np.uint32)
    span_idx = np.array([j for _, j in call], dtype=np.uint32)
    n_tokens = np.array([w.spans_of(s)[1][j] for s, j in call], dtype=np.uint32)
    return slots, span_idx, n_tokens


def host_span(w, s, j):
    v = workloads.span_values(w, s, j)
    return bits16(v) if w.src_dtype == 0 else bits32(v)


def run_oracle(w, table=None, keep_pool=False):
    """register -> write (per the workload's call schedule) -> plan -> gather everything."""
    pool = OraclePool(PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0, pool.rc
    res = {"rc": []}
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        res["rc"].append(pool.register_samples(*register_args(w, samples)))
        slots, span_idx, n_tokens = write_args(w, call)
        srcs = [host_span(w, s, j) for s, j in call]
        res["rc"].append(pool.write_embeddings(slots, span_idx, n_tokens, srcs, w.src_dtype))
    rc, plan = pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), PlanConfig(**plan_config_fields(w)))
    res["rc"].append(rc)
    assert rc == 0, rc
    res["plan"] = plan.arrays()
    n_mb, total, _ = plan.summary()
    if table is None:
        table = bits16(workloads.embed_table(w))
    out = np.full((total, w.hidden), 0xFFFF, dtype=np.uint16)
    cu = np.full(len(w.plan_order) + n_mb, -1, dtype=np.int32)
    pos = np.full(total, -1, dtype=np.int32)
    res["rc"].append(pool.gather_packed(plan, 0, n_mb, table, out, cu, pos))
    res.update(out=out, cu_seqlens=cu, position_ids=pos, table=table, status=pool.status())
    res["span_pages"] = {(s, j): pool.span_pages(s, j)[1] for call in w.write_calls for s, j in call}
    if keep_pool:
        res["pool"], res["plan_handle"] = pool, plan
    else:
        plan.destroy()
        pool.destroy()
    return res
