"""Feeds the CUDA library (through its Python binding) the same call sequence tests/harness.py feeds the
oracle.  Marshalling only."""
import numpy as np
import torch

import workloads
from harness import pool_config_fields, plan_config_fields, register_args, write_args, bits16, bits32
from paper_2606_23087_b200 import binding as fp


def cuda_stream():
    return torch.cuda.current_stream().cuda_stream


def device_span(w, s, j):
    return workloads.span_values(w, s, j, device="cuda")


def host_bits(t):
    return bits16(t) if t.dtype == torch.bfloat16 else bits32(t)


class CudaRun:
    """register -> write -> plan -> gather over a workload, keeping device buffers alive."""

    def __init__(self, w, caller_owned_memory=False, max_samples=None, tuning=None):
        self.w = w
        self.keep = []
        f = pool_config_fields(w, max_samples=max_samples)
        hbm_ptr = host_ptr = 0
        if caller_owned_memory:
            if w.hbm_pages:
                self.hbm = torch.full((w.hbm_pages * w.page_bytes + 256,), 0xFF, dtype=torch.uint8, device="cuda")
                hbm_ptr = (self.hbm.data_ptr() + 255) // 256 * 256
        self.pool = fp.Pool(fp.PoolConfig(**f), hbm_base=hbm_ptr, host_base=host_ptr)
        assert self.pool.rc == 0, fp.STATUS.get(self.pool.rc)
        if tuning:
            assert self.pool.set_tuning(**tuning) == 0
        self.rc = []
        self.srcs = {}

    def register(self, samples):
        slots, seq_len, n_spans, pos, tok, ids = register_args(self.w, samples)
        d_ids = torch.from_numpy(ids).cuda()
        self.keep.append(d_ids)
        rc = self.pool.register_samples(slots, seq_len, n_spans, pos, tok, d_ids.data_ptr(), cuda_stream())
        self.rc.append(rc)
        return rc

    def write(self, call, keep_src=True):
        slots, span_idx, n_tokens = write_args(self.w, call)
        srcs = [device_span(self.w, s, j) for s, j in call]
        if keep_src:
            for c, t in zip(call, srcs):
                self.srcs[c] = t
        else:
            self.keep.append(srcs)
        rc = self.pool.write_embeddings(slots, span_idx, n_tokens, [t.data_ptr() for t in srcs], self.w.src_dtype,
                                        cuda_stream())
        self.rc.append(rc)
        return rc

    def run_schedule(self):
        for call in self.w.write_calls:
            samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
            self.register(samples)
            self.write(call)

    def plan(self, order=None, flags=0):
        order = self.w.plan_order if order is None else order
        rc, plan = self.pool.plan_microbatches(np.asarray(order, dtype=np.uint32),
                                               fp.PlanConfig(**plan_config_fields(self.w, flags)), cuda_stream())
        self.rc.append(rc)
        self.plan_handle = plan
        return rc, plan

    def gather_all(self, table=None, n_samples=None):
        plan = self.plan_handle
        n_mb, total, _ = plan.summary()
        if table is None:
            table = workloads.embed_table(self.w, device="cuda")
        self.table = table
        n = len(self.w.plan_order) if n_samples is None else n_samples
        out = torch.full((total, self.w.hidden), -1, dtype=torch.int16, device="cuda")  # 0xFFFF poison
        cu = torch.full((n + n_mb,), -1, dtype=torch.int32, device="cuda")
        pos = torch.full((total,), -1, dtype=torch.int32, device="cuda")
        rc = self.pool.gather_packed(plan, 0, n_mb, table.data_ptr(), table.shape[0], out.data_ptr(), cu.data_ptr(),
                                     pos.data_ptr(), cuda_stream())
        self.rc.append(rc)
        torch.cuda.synchronize()
        return rc, out, cu, pos

    def close(self):
        torch.cuda.synchronize()
        if getattr(self, "plan_handle", None):
            self.plan_handle.destroy()
        self.pool.destroy()


def run_cuda(w, caller_owned_memory=False, tuning=None):
    r = CudaRun(w, caller_owned_memory, tuning=tuning)
    r.run_schedule()
    rc, plan = r.plan()
    assert rc == 0, fp.STATUS.get(rc)
    res = {"plan": plan.arrays()}
    rc, out, cu, pos = r.gather_all()
    res.update(rc=r.rc, out=out.cpu().numpy().view(np.uint16), cu_seqlens=cu.cpu().numpy(),
               position_ids=pos.cpu().numpy(), status=r.pool.status(), table=bits16(r.table))
    res["span_pages"] = {(s, j): r.pool.span_pages(s, j)[1] for call in w.write_calls for s, j in call}
    res["srcs"] = {c: host_bits(t) for c, t in r.srcs.items()}
    res["stats"] = r.pool.stats()
    r.close()
    return res
