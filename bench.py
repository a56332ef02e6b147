#!/usr/bin/env python
"""Benchmark of the unified-memory-pool hot path on B200.

A step is one pass of the whole path over one batch of the "7B-class image mix" workload
(512 samples, hidden 3584, 2 MiB pages, pool 80 % HBM / 20 % pinned host): for each of the 16 producer
calls register the samples and scatter their embeddings into pages; plan the microbatches (Algorithm 1);
gather every packed microbatch; free the samples.  `value` is the step's algorithmic bytes
(4H per vision token written + 4H per packed token assembled) over its device time, inputs resident in HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--all-hbm] [--samples S]

One JSON line on stdout (rank 0).  `--impl reference` times the CPU oracle, as it stands, on a bounded
sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
for p in (ROOT, os.path.join(ROOT, "tests")):
    if p not in sys.path:
        sys.path.insert(0, p)

METRIC = "packed-microbatch assembly throughput (producer scatter + plan + packed gather + free)"
UNIT = "GB/s"
CPU_SAMPLE = 256         # samples of the workload the oracle is timed on (about 10-30 s of CPU work)
# dram__bytes_read.sum + dram__bytes_write.sum over algorithmic bytes for one k_gather launch, from the ncu capture
# on the first 64 samples of this workload, all pages in HBM (4.592 GB of DRAM traffic / 4.698 GB algorithmic);
# traffic grows in proportion to the tokens assembled, so a full launch is this ratio times its algorithmic bytes
NCU_TRAFFIC_RATIO_GATHER = 0.977


def algorithmic_bytes(w):
    """Bytes the method must move in one step: write 4H per vision token (bf16 source; 6H from fp32),
    gather 4H per packed token."""
    per_vis = (2 if w.src_dtype == 0 else 4) * w.hidden + 2 * w.hidden
    return w.total_vision_tokens * per_vis, w.total_tokens * 4 * w.hidden


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# CPU oracle arm (cpu_baseline, and --impl reference)
# ---------------------------------------------------------------------------------------------
def oracle_setup(name, n_samples, all_hbm):
    import torch
    import workloads
    from harness import bits16, bits32, pool_config_fields, plan_config_fields, register_args, write_args
    from oracle import OraclePool, PlanConfig, PoolConfig
    w = workloads.make_workload(name, n_samples=n_samples, all_hbm=all_hbm)
    dev = "cuda" if torch.cuda.is_available() else "cpu"   # inputs only: the generator is device independent
    conv = bits16 if w.src_dtype == 0 else bits32
    srcs = {c: conv(workloads.span_values(w, c[0], c[1], device=dev)) for call in w.write_calls for c in call}
    table = bits16(workloads.embed_table(w, device=dev))
    calls = []
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        calls.append((register_args(w, samples), write_args(w, call), [srcs[c] for c in call]))
    pool = OraclePool(PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    out = np.empty((w.total_tokens, w.hidden), dtype=np.uint16)
    cu = np.empty(w.n_samples * 2 + 8, dtype=np.int32)
    pos = np.empty(w.total_tokens, dtype=np.int32)
    pcfg = PlanConfig(**plan_config_fields(w))
    order = np.asarray(w.plan_order, dtype=np.uint32)

    def step():
        for reg, wr, s in calls:
            assert pool.register_samples(*reg) == 0
            assert pool.write_embeddings(*wr, s, w.src_dtype) == 0
        rc, plan = pool.plan_microbatches(order, pcfg)
        assert rc == 0
        n_mb = plan.summary()[0]
        assert pool.gather_packed(plan, 0, n_mb, table, out, cu, pos) == 0
        plan.destroy()
        assert pool.free(order) == 0
    return w, step


def time_oracle_gather_threads(name, n_samples, all_hbm, reps=2):
    """The oracle's assembly alone, as it stands, once on one core and once with the microbatches split over all
    cores this process may use (one thread per contiguous range of microbatches; ctypes releases the GIL)."""
    import concurrent.futures
    import torch
    import workloads
    from harness import bits16, bits32, pool_config_fields, plan_config_fields, register_args, write_args
    from oracle import OraclePool, PlanConfig, PoolConfig
    w = workloads.make_workload(name, n_samples=n_samples, all_hbm=all_hbm)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    conv = bits16 if w.src_dtype == 0 else bits32
    table = bits16(workloads.embed_table(w, device=dev))
    pool = OraclePool(PoolConfig(**pool_config_fields(w)))
    assert pool.rc == 0
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        assert pool.register_samples(*register_args(w, samples)) == 0
        srcs = [conv(workloads.span_values(w, s, j, device=dev)) for s, j in call]
        assert pool.write_embeddings(*write_args(w, call), srcs, w.src_dtype) == 0
    rc, plan = pool.plan_microbatches(np.asarray(w.plan_order, dtype=np.uint32), PlanConfig(**plan_config_fields(w)))
    assert rc == 0
    a = plan.arrays()
    n_mb = int(a["n_mb"])
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    tok = np.concatenate([[0], np.cumsum(a["mb_tokens"].astype(np.int64))])

    def ranges(parts):
        cuts = sorted({int(np.searchsorted(tok, tok[-1] * k / parts)) for k in range(parts + 1)} | {0, n_mb})
        return [(b, e) for b, e in zip(cuts[:-1], cuts[1:]) if e > b]

    def run(parts):
        bufs = []
        for b, e in ranges(parts):
            rows = int(tok[e] - tok[b])
            n_s = int(a["mb_sample_off"][e] - a["mb_sample_off"][b])
            bufs.append((b, e, np.empty((rows, w.hidden), np.uint16), np.empty(n_s + (e - b), np.int32), np.empty(rows, np.int32)))
        best = None
        for _ in range(reps):
            t0 = time.perf_counter()
            if len(bufs) == 1:
                b, e, o, c, p_ = bufs[0]
                assert pool.gather_packed(plan, b, e, table, o, c, p_) == 0
            else:
                with concurrent.futures.ThreadPoolExecutor(len(bufs)) as ex:
                    rcs = list(ex.map(lambda t: pool.gather_packed(plan, t[0], t[1], table, t[2], t[3], t[4]), bufs))
                assert all(r == 0 for r in rcs)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        return best, len(bufs)

    gb = w.total_tokens * 4 * w.hidden
    t1, _ = run(1)
    tn, used = run(min(cores, n_mb))
    plan.destroy()
    pool.destroy()
    return {"gather_1_core_gbs": gb / t1 / 1e9, "gather_all_cores_gbs": gb / tn / 1e9, "gather_threads": used,
            "cores_available": cores}


def time_oracle(name, n_samples, all_hbm, steps, warmup):
    w, step = oracle_setup(name, n_samples, all_hbm)
    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    wb, gb = algorithmic_bytes(w)
    return {"value": (wb + gb) / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"first {n_samples} of the workload's samples ({w.total_tokens} packed tokens), whole step, "
                      f"{dt * 1e3:.0f} ms per step, {steps} step(s)",
            "tokens_per_s": w.total_tokens / dt, "ms_per_step": dt * 1e3}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n = min(CPU_SAMPLE, args.samples or CPU_SAMPLE)
    r = time_oracle(args.workload, n, args.all_hbm, max(1, args.steps), min(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": workload_label(args), "cpu_sample_samples": n},
        "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": 1, "kind": "oracle", "sample": r["sample"]},
        "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "tokens_per_s": r["tokens_per_s"], "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_label(args, all_hbm=None):
    all_hbm = args.all_hbm if all_hbm is None else all_hbm
    split = {"image_mix_7b": "pool 80% HBM / 20% pinned host", "host_tier_stress": "pool 50% HBM / 50% pinned host, tiers interleaved"}
    tier = "all pages in HBM" if (all_hbm or args.workload not in split) else split[args.workload]
    n = f", first {args.samples} samples" if args.samples else ""
    if args.workload != "image_mix_7b":
        return f"{args.workload} ({tier}){n}"
    return f"{args.workload}: 512 samples, 1-4 images, hidden 3584, 2 MiB pages, {tier}, budget 32768{n}"


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------
class DeviceJob:
    """All device state of one rank: pool, resident inputs, outputs, and the step function."""

    def __init__(self, args, all_hbm):
        import torch
        import workloads
        from harness import pool_config_fields, plan_config_fields, register_args, write_args
        from paper_2606_23087_b200 import binding as fp
        self.torch, self.fp = torch, fp
        w = workloads.make_workload(args.workload, n_samples=args.samples, all_hbm=all_hbm, id_skew=getattr(args, "id_skew", "uniform"))
        if getattr(args, "bind_order", "workload") == "identity":
            w.bind_order = 0      # virtual page k lives in frame k: a span's consecutive pages are contiguous in the slab
        self.w = w
        self.pool = fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
        if self.pool.rc != 0:
            raise fp.FlowpoolError(self.pool.rc, "pool_create")
        apply_tuning(self.pool, args)
        self.table = workloads.embed_table(w, device="cuda")
        self.calls = []
        for call in w.write_calls:
            samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
            reg = register_args(w, samples)
            ids = torch.from_numpy(reg[5]).cuda()
            srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]
            self.calls.append({"reg": reg[:5], "ids": ids, "wr": write_args(w, call), "srcs": srcs,
                               "ptrs": [t.data_ptr() for t in srcs]})
        self.out = torch.empty((w.total_tokens, w.hidden), dtype=torch.bfloat16, device="cuda")
        self.cu = torch.empty((w.n_samples * 2 + 8,), dtype=torch.int32, device="cuda")
        self.pos = torch.empty((w.total_tokens,), dtype=torch.int32, device="cuda")
        self.order = np.asarray(w.plan_order, dtype=np.uint32)
        self.pcfg = fp.PlanConfig(**plan_config_fields(w))
        self.plan_ms = []

    def check(self, rc, where):
        if rc != 0:
            raise self.fp.FlowpoolError(rc, where)

    def fits_l2(self):
        """True when the bytes one step touches (sources, pool pages, table rows read, output) could sit in L2."""
        wb, gb = algorithmic_bytes(self.w)
        return wb + gb < (512 << 20)

    def step(self, before_write=None, after_gather=None, bufs=None, before_gather=None, after_write=None):
        out, cu, pos = bufs or (self.out, self.cu, self.pos)
        st = self.torch.cuda.current_stream().cuda_stream
        pool = self.pool
        for i, c in enumerate(self.calls):
            if before_write:
                before_write(i, c)
            self.check(pool.register_samples(*c["reg"], c["ids"].data_ptr(), st), "pool_register_samples")
            self.check(pool.write_embeddings(*c["wr"], c["ptrs"], self.w.src_dtype, st), "pool_write_embeddings")
            if after_write:
                after_write(i, c)
        t0 = time.perf_counter()
        rc, plan = pool.plan_microbatches(self.order, self.pcfg, st)
        self.check(rc, "pool_plan_microbatches")
        self.plan_ms.append((time.perf_counter() - t0) * 1e3)   # includes waiting for the writes queued before it
        n_mb = plan.summary()[0]
        if before_gather:
            before_gather()
        self.check(pool.gather_packed(plan, 0, n_mb, self.table.data_ptr(), self.w.vocab, out.data_ptr(),
                                      cu.data_ptr(), pos.data_ptr(), st), "pool_gather_packed")
        if after_gather:
            after_gather()
        self.check(pool.free(self.order, st), "pool_free")
        plan.destroy()
        return n_mb

    # -- which bytes of a step land on host-tier pages -------------------------------------------------------
    # The free ring is a FIFO over global page indices (indices below hbm_pages are HBM frames): a write call's spans
    # pop consecutive entries in argument order, pool_free pushes a sample's pages back in argument order, spans by
    # index, pages by ordinal.  The pool is barely larger than one batch, so the ring rotates from step to step and the
    # share of a batch that lands on host-tier pages differs per step.  The benchmark follows the ring on the host
    # (bookkeeping only) to know, for every timed step, how many bytes crossed the host link; the model is checked
    # against the pool's own ring afterwards.
    def ring_model_reset(self):
        import collections
        self.model_ring = collections.deque(int(x) for x in self.pool.ring())   # synchronises: outside timed regions

    def ring_model_step(self):
        """Host-tier vision bytes of one step (write everything, then free everything in plan order)."""
        w, ring = self.w, self.model_ring
        host_b, pages_of = 0, {}
        for call in w.write_calls:
            for s, j in call:
                nbytes = int(w.spans_of(s)[1][j]) * w.row_bytes
                got = [ring.popleft() for _ in range(-(-nbytes // w.page_bytes))]
                pages_of[(s, j)] = got
                for o, g in enumerate(got):
                    if g >= w.hbm_pages:
                        host_b += min(w.page_bytes, nbytes - o * w.page_bytes)
        for s in self.order:
            for j in range(int(w.n_spans[int(s)])):
                ring.extend(pages_of[(int(s), j)])
        return host_b

    def ring_model_matches(self):
        return [int(x) for x in self.pool.ring()] == list(self.model_ring)

    def close(self):
        self.torch.cuda.synchronize()
        self.pool.destroy()


def apply_tuning(pool, args):
    """--tuning key=value,...: launch-geometry knobs of the library (pool_set_tuning), for sweeps."""
    spec = getattr(args, "tuning", None)
    if spec:
        rc = pool.set_tuning(**{k: int(v) for k, v in (kv.split("=") for kv in spec.split(","))})
        if rc != 0:
            raise SystemExit(f"pool_set_tuning({spec}) -> {rc}")


def measure_host_link(torch, nbytes=1 << 30, reps=5):
    """Host-link reference rates: plain cudaMemcpyAsync between pinned host memory and the device, best of reps, one
    direction at a time, and one copy each way at the same time on two streams (what the copy engines get when the
    link is used in both directions at once)."""
    try:
        h = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
        d = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        h2 = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
        d2 = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    except RuntimeError:
        return None
    res = {}
    for name, (dst, src) in (("h2d_gbs", (d, h)), ("d2h_gbs", (h, d))):
        best = 0.0
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            dst.copy_(src, non_blocking=True)
            e1.record()
            torch.cuda.synchronize()
            best = max(best, nbytes / e0.elapsed_time(e1) / 1e6)
        res[name] = best
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    best = None
    for _ in range(reps):
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        with torch.cuda.stream(s1):
            ev[0].record(); d.copy_(h, non_blocking=True); ev[1].record()
        with torch.cuda.stream(s2):
            ev[2].record(); h2.copy_(d2, non_blocking=True); ev[3].record()
        torch.cuda.synchronize()
        a, b = nbytes / ev[0].elapsed_time(ev[1]) / 1e6, nbytes / ev[2].elapsed_time(ev[3]) / 1e6
        if best is None or a + b > best[0] + best[1]:
            best = (a, b)
    res["both_ways_h2d_gbs"], res["both_ways_d2h_gbs"] = best
    return res


def max_over_ranks(ms, dist, device="cuda"):
    """A multi-rank time is the slowest rank's."""
    if dist is None:
        return ms
    import torch
    if dist.get_backend() != "nccl":
        device = "cpu"
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_rank, world, ms):
    """Whole-job GB/s: every rank moved bytes_per_rank in the (max-over-ranks) step time."""
    return world * bytes_per_rank / ms / 1e6


def timed_steps(job, steps, warmup, dist):
    torch = job.torch
    for _ in range(warmup):
        job.step()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    job.ring_model_reset()
    job.host_bytes_per_step = [job.ring_model_step() for _ in range(steps)] if job.w.host_pages else [0] * steps
    job.pool.profile_read()
    job.pool.profile_enable(True)
    launches0 = job.pool.stats()["gpu_launches"]
    job.plan_ms.clear()
    n_mb = 0
    if job.fits_l2():
        # a working set that could stay in the 126 MB L2: every step is timed on its own and a 512 MiB scrub
        # between steps evicts it (the scrub is outside the timed regions)
        scrub = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
        total = 0.0
        for i in range(steps):
            scrub.fill_(i & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            n_mb = job.step()
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
        ms = total / steps
        del scrub
    else:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            n_mb = job.step()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
    prof = job.pool.profile_read()
    job.pool.profile_enable(False)
    launches = job.pool.stats()["gpu_launches"] - launches0
    job.ring_ok = job.ring_model_matches() if job.w.host_pages else True
    job.plan_ms_in_step = float(np.median(job.plan_ms)) if job.plan_ms else None
    if dist:
        ms = max_over_ranks(ms, dist)
        dist.barrier()
    torch.cuda.synchronize()
    return ms, prof, launches, n_mb


def phase_breakdown(job, reps=3):
    """Device time of each phase of a step, from extra (untimed-region) steps with a synchronize between phases:
    register+write (all producer calls), plan, gather, free.  Median over `reps`."""
    torch, pool, w = job.torch, job.pool, job.w
    st = torch.cuda.current_stream().cuda_stream
    acc = {"write": [], "plan": [], "gather": [], "free": []}

    def timed(fn):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        r = fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), r

    for _ in range(reps):
        def do_write():
            for c in job.calls:
                job.check(pool.register_samples(*c["reg"], c["ids"].data_ptr(), st), "register")
                job.check(pool.write_embeddings(*c["wr"], c["ptrs"], w.src_dtype, st), "write")
        ms, _ = timed(do_write)
        acc["write"].append(ms)
        ms, (rc, plan) = timed(lambda: pool.plan_microbatches(job.order, job.pcfg, st))
        job.check(rc, "plan")
        acc["plan"].append(ms)
        n_mb = plan.summary()[0]
        ms, rc = timed(lambda: pool.gather_packed(plan, 0, n_mb, job.table.data_ptr(), w.vocab, job.out.data_ptr(),
                                                  job.cu.data_ptr(), job.pos.data_ptr(), st))
        job.check(rc, "gather")
        acc["gather"].append(ms)
        ms, rc = timed(lambda: pool.free(job.order, st))
        job.check(rc, "free")
        acc["free"].append(ms)
        plan.destroy()
    return {k: float(np.median(v)) for k, v in acc.items()}


def kernel_breakdown(job, prof, steps):
    """Per-kernel-class time per step and achieved bandwidth against the bytes that class moves."""
    w = job.w
    host_b = float(np.mean(job.host_bytes_per_step))   # what the timed steps actually put on host-tier pages, per step
    vis_b = w.total_vision_tokens * w.row_bytes
    tok_b = w.total_tokens * w.row_bytes
    src_mult = 1 if w.src_dtype == 0 else 2
    moved = {
        "gather_device": 2 * (tok_b - host_b), "gather_host": 2 * host_b,
        "scatter_device": (1 + src_mult) * (vis_b - host_b), "scatter_host": (1 + src_mult) * host_b,
    }
    out = {}
    for k, v in prof.items():
        if k not in moved:
            continue
        ms = v["ms"] / steps
        out[k] = {"ms_per_step": ms, "launches_per_step": v["launches"] / steps, "bytes_per_step": moved[k],
                  "gbs": (moved[k] / ms / 1e6) if ms > 0 else None}
    return out, host_b


def run_e2e(job, steps):
    """The same step through host buffers: every producer call's embeddings and ids come from pinned host
    memory (H2D inside the timed region) and the packed result goes back to pinned host memory (D2H)."""
    torch = job.torch
    w = job.w
    try:
        # one contiguous pinned buffer (and one device buffer) per producer call, the spans one after the other: a
        # call's embeddings cross the link as one copy (many small copies lose the link to a large copy going the
        # other way: 4 GiB each way moves at 91 GB/s in all as single copies, at 56 GB/s with 1 MiB pieces)
        host_src, dev_src = [], []
        for c in job.calls:
            sizes = [t.numel() for t in c["srcs"]]
            h = torch.empty(sum(sizes), dtype=c["srcs"][0].dtype, pin_memory=True)
            d = torch.empty(sum(sizes), dtype=c["srcs"][0].dtype, device="cuda")
            o = 0
            ptrs = []
            for t, nel in zip(c["srcs"], sizes):
                h[o:o + nel].copy_(t.reshape(-1))
                ptrs.append(d.data_ptr() + o * d.element_size())
                o += nel
            host_src.append(h); dev_src.append(d)
            c["ptrs_resident"], c["ptrs"] = c["ptrs"], ptrs      # the step reads the staged copies
        host_ids = [torch.empty(c["ids"].shape, dtype=c["ids"].dtype, pin_memory=True).copy_(c["ids"]) for c in job.calls]
        host_out = torch.empty(job.out.shape, dtype=job.out.dtype, pin_memory=True)
        host_cu = torch.empty(job.cu.shape, dtype=job.cu.dtype, pin_memory=True)
        host_pos = torch.empty(job.pos.shape, dtype=job.pos.dtype, pin_memory=True)
    except RuntimeError as e:
        for c in job.calls:
            if "ptrs_resident" in c:
                c["ptrs"] = c.pop("ptrs_resident")
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0, "error": str(e)[:120]}
    h2d = sum(t.numel() * t.element_size() for t in host_src) + sum(t.numel() * 4 for t in host_ids)
    d2h = host_out.numel() * 2 + host_cu.numel() * 4 + host_pos.numel() * 4

    def before_write(i, c):
        dev_src[i].copy_(host_src[i], non_blocking=True)
        c["ids"].copy_(host_ids[i], non_blocking=True)

    def after_gather():
        host_out.copy_(job.out, non_blocking=True)
        host_cu.copy_(job.cu, non_blocking=True)
        host_pos.copy_(job.pos, non_blocking=True)

    job.step(before_write, after_gather)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        job.step(before_write, after_gather)
    e1.record()
    torch.cuda.synchronize()
    ms_serial = e0.elapsed_time(e1) / steps
    # the round trip is only worth something if the bytes came back right: spot-check against the device copy
    ok = bool(torch.equal(host_out[:64].view(torch.int16), job.out[:64].cpu().view(torch.int16)))

    # The same steps, pipelined the way a training loop would run them.  Result: the packed output of step k goes back
    # to the host on a copy stream while step k+1 runs (two result buffers; a buffer is reused only after its copy-out
    # has finished).  Inputs: every producer call has a device buffer of its own, so the inputs of call i of step k+1
    # come in on a third stream as soon as the scatter of call i of step k has read that buffer; the producer call
    # waits only for its own inputs.  The link is full duplex: inputs and host-tier reads go one way, the result and
    # host-tier writes the other.
    ms_pipe = None
    try:
        bufs = [(job.out, job.cu, job.pos),
                (torch.empty_like(job.out), torch.empty_like(job.cu), torch.empty_like(job.pos))]
        copy_stream, h2d_stream = torch.cuda.Stream(), torch.cuda.Stream()
        main = torch.cuda.current_stream()
        done = [None, None]
        n_calls = len(job.calls)
        loaded, consumed = [None] * n_calls, [None] * n_calls

        def prefetch(i):
            if consumed[i] is not None:
                h2d_stream.wait_event(consumed[i])           # the scatter that last read this device buffer
            with torch.cuda.stream(h2d_stream):
                dev_src[i].copy_(host_src[i], non_blocking=True)
                job.calls[i]["ids"].copy_(host_ids[i], non_blocking=True)
                loaded[i] = torch.cuda.Event()
                loaded[i].record(h2d_stream)

        def inputs_ready(i, c):
            main.wait_event(loaded[i])

        def inputs_consumed(i, c):
            consumed[i] = torch.cuda.Event()
            consumed[i].record(main)
            prefetch(i)                                      # the same call of the next step

        def pipelined(n):
            for k in range(n):
                b = k % 2

                def buffer_free(b=b):   # the result buffer is needed by the assembly only, not by the writes before it
                    if done[b] is not None:
                        main.wait_event(done[b])

                def copy_out(b=b):
                    ready = torch.cuda.Event()
                    ready.record(main)
                    copy_stream.wait_event(ready)
                    with torch.cuda.stream(copy_stream):
                        host_out.copy_(bufs[b][0], non_blocking=True)
                        host_cu.copy_(bufs[b][1], non_blocking=True)
                        host_pos.copy_(bufs[b][2], non_blocking=True)
                        done[b] = torch.cuda.Event()
                        done[b].record(copy_stream)
                job.step(inputs_ready, copy_out, bufs=bufs[b], before_gather=buffer_free, after_write=inputs_consumed)
            main.wait_stream(copy_stream)

        for i in range(n_calls):
            prefetch(i)
        pipelined(2)
        torch.cuda.synchronize()
        n_pipe = max(4, 2 * steps)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record()
        pipelined(n_pipe)
        p1.record()
        torch.cuda.synchronize()
        ms_pipe = p0.elapsed_time(p1) / n_pipe
        ok = ok and bool(torch.equal(host_out[-64:].view(torch.int16), bufs[(n_pipe - 1) % 2][0][-64:].cpu().view(torch.int16)))
        ok = ok and bool(torch.equal(host_out[:64].view(torch.int16), bufs[(n_pipe - 1) % 2][0][:64].cpu().view(torch.int16)))
    except RuntimeError:
        ms_pipe = None
    for c in job.calls:
        c["ptrs"] = c.pop("ptrs_resident")
    del dev_src
    wb, gb = algorithmic_bytes(w)
    ms = min(ms_serial, ms_pipe) if ms_pipe else ms_serial
    return {"value": (wb + gb) / ms / 1e6, "unit": UNIT, "ms_per_step": ms, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": steps, "readback_matches": ok,
            "serial_ms_per_step": ms_serial, "pipelined_ms_per_step": ms_pipe,
            "note": "value = steady state with the result copy-out of step k and the inputs of step k+1 each on a copy stream of their own beside the step's kernels"}


def backbone_side(job, reps=3):
    """Backbone-side outputs on the job's batch (device-resident, timed with CUDA events on the launching stream):
    the padded assembly with positions, ids, labels and mask, and the ordered table gradient."""
    import workloads
    torch, pool, w = job.torch, job.pool, job.w
    st = torch.cuda.current_stream().cuda_stream
    for c in job.calls:
        job.check(pool.register_samples(*c["reg"], c["ids"].data_ptr(), st), "register")
        job.check(pool.write_embeddings(*c["wr"], c["ptrs"], w.src_dtype, st), "write")
    items = [(s, j, workloads.span_grid(w, s, j)) for s in range(w.n_samples) for j in range(int(w.n_spans[s]))]
    items = [it for it in items if it[2] is not None]
    job.check(pool.set_span_grids([s for s, _, _ in items], [j for _, j, _ in items], [g for _, _, g in items], st), "pool_set_span_grids")
    rc, plan = pool.plan_microbatches(job.order, job.pcfg, st)
    job.check(rc, "plan")
    a = plan.arrays()
    n_mb, L, H = int(a["n_mb"]), w.budget_L, w.hidden
    per_call = max(1, job.out.shape[0] // L)       # microbatches whose padded rows fit the job's output buffer
    rows_cap = per_call * L
    out = job.out if job.out.shape[0] >= rows_cap else torch.empty((rows_cap, H), dtype=torch.bfloat16, device="cuda")
    cu = torch.empty((w.n_samples + 2 * n_mb + 8,), dtype=torch.int32, device="cuda")
    pos3 = torch.empty((3 * rows_cap,), dtype=torch.int32, device="cuda")
    ids = torch.empty((rows_cap,), dtype=torch.int32, device="cuda")
    labels = torch.empty((rows_cap,), dtype=torch.int32, device="cuda")
    mask = torch.empty((rows_cap,), dtype=torch.uint8, device="cuda")

    def timed(fn):
        best = []
        for _ in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            best.append(e0.elapsed_time(e1))
        return float(np.median(best[1:]))

    def padded_all():
        for b in range(0, n_mb, per_call):
            e = min(n_mb, b + per_call)
            job.check(pool.gather_padded(plan, b, e, job.table.data_ptr(), w.vocab, 0, out.data_ptr(), cu.data_ptr(),
                                         pos3.data_ptr(), ids.data_ptr(), labels.data_ptr(), mask.data_ptr(), st), "pool_gather_padded")

    def packed_all():
        job.check(pool.gather_packed(plan, 0, n_mb, job.table.data_ptr(), w.vocab, job.out.data_ptr(), job.cu.data_ptr(),
                                     job.pos.data_ptr(), st), "pool_gather_packed")

    ms_packed = timed(packed_all)
    ms_padded = timed(padded_all)
    # every rank's share of the zig-zag deal: one list call per rank, against one range call per microbatch
    rank_lists = [[int(j) for j in a["rank_mbs"][a["rank_mb_off"][k]:a["rank_mb_off"][k + 1]]] for k in range(w.n_ranks_N)]
    mb_rows = np.concatenate([[0], np.cumsum(a["mb_tokens"].astype(np.int64))])

    def by_rank_lists():
        base = 0
        for lst in rank_lists:
            if lst:
                job.check(pool.gather_list(plan, lst, job.table.data_ptr(), w.vocab, job.out[base:].data_ptr(), job.cu.data_ptr(),
                                           job.pos.data_ptr(), st), "pool_gather_list")
            base += int(sum(mb_rows[j + 1] - mb_rows[j] for j in lst))

    def by_microbatch():
        for j in range(n_mb):
            job.check(pool.gather_packed(plan, j, j + 1, job.table.data_ptr(), w.vocab, job.out[int(mb_rows[j]):].data_ptr(),
                                         job.cu.data_ptr(), job.pos.data_ptr(), st), "pool_gather_packed")

    ms_rank_lists = timed(by_rank_lists)
    ms_per_mb = timed(by_microbatch)
    gather_bytes = w.total_tokens * 4 * H
    pad_rows = n_mb * L - w.total_tokens
    padded_bytes = w.total_tokens * 4 * H + pad_rows * 2 * H + n_mb * L * 21   # rows read+written, zero rows, 21 index bytes per row
    # table gradient: the assembled rows stand in for the gradient (bf16 values of unit scale), packed layout
    packed_all()
    grad_table = torch.zeros((w.vocab, H), dtype=torch.float32, device="cuda")
    pool.profile_read()
    pool.profile_enable(True)
    ms_grad_call = timed(lambda: job.check(pool.embed_grad(plan, 0, n_mb, False, job.out.data_ptr(), grad_table.data_ptr(),
                                                           w.vocab, st), "pool_embed_grad"))
    prof = pool.profile_read()["embed_grad"]
    pool.profile_enable(False)
    ms_grad_kernel = prof["ms"] / max(1, prof["launches"])
    text_rows = w.total_tokens - w.total_vision_tokens
    grad_bytes = text_rows * 10 * H + w.total_tokens * 8       # bf16 row in, fp32 row read and written; row ids written and read
    all_ids = np.concatenate([workloads.input_ids(w, s) for s in range(w.n_samples)])
    distinct = int(len(np.unique(all_ids[all_ids != w.placeholder_id])))
    floor_bytes = text_rows * 2 * H + distinct * 8 * H         # every gradient row once, every touched table row once
    peak = measured_peak()[0]
    job.check(pool.free(job.order, st), "free")
    plan.destroy()
    torch.cuda.synchronize()
    return {
        "gather_packed_ms": ms_packed,
        "gather_rank_lists": {"ms": ms_rank_lists, "calls": len(rank_lists), "gbs": gather_bytes / ms_rank_lists / 1e6,
                              "per_microbatch_range_calls_ms": ms_per_mb, "per_microbatch_calls": n_mb,
                              "per_microbatch_gbs": gather_bytes / ms_per_mb / 1e6},
        "gather_padded": {"ms": ms_padded, "calls": -(-n_mb // per_call), "padding_rows": int(pad_rows), "algorithmic_bytes": int(padded_bytes),
                          "gbs": padded_bytes / ms_padded / 1e6, "frac_of_measured_peak": padded_bytes / ms_padded / 1e6 / peak,
                          "outputs": "embeds, cu_seqlens, 3-component positions, ids, labels, loss mask"},
        "embed_grad": {"ms_call": ms_grad_call, "ms_kernel": ms_grad_kernel, "text_rows": int(text_rows), "algorithmic_bytes": int(grad_bytes),
                       "gbs": grad_bytes / ms_grad_kernel / 1e6, "frac_of_measured_peak": grad_bytes / ms_grad_kernel / 1e6 / peak,
                       "bound": "hbm", "ids": w.id_skew, "distinct_ids": distinct, "floor_bytes": int(floor_bytes),
                       "note": "algorithmic_bytes = 10H per text row (bf16 gradient row in, fp32 table row read and written); "
                               "floor_bytes = each gradient row and each touched table row once; frequent ids keep their sum in "
                               "registers, so skewed ids move fewer bytes than the 10H model"},
    }


def short_pass(args, name, all_hbm, steps=3):
    """One short timed pass of the whole step on another configuration, with the per-kernel-class figures."""
    import copy
    import gc
    a = copy.copy(args)
    a.workload, a.samples, a.all_hbm = name, None, all_hbm
    job = DeviceJob(a, all_hbm)
    ms, prof, launches, n_mb = timed_steps(job, steps, 3, None)
    kern, host_b = kernel_breakdown(job, prof, steps)
    phases = phase_breakdown(job, reps=2)
    wb, gb = algorithmic_bytes(job.w)
    peak = measured_peak()[0]
    g = kern["gather_device"] if kern["gather_device"]["ms_per_step"] > 0 else kern["gather_host"]
    sc = kern["scatter_device"] if kern["scatter_device"]["ms_per_step"] > 0 else kern["scatter_host"]
    res = {"workload": workload_label(a), "step_ms": ms, "value": (wb + gb) / ms / 1e6, "unit": UNIT, "tokens_per_s": job.w.total_tokens / ms * 1e3,
           "packed_tokens": job.w.total_tokens, "microbatches": n_mb, "gpu_launches_per_step": launches / steps,
           "gather_gbs": g["gbs"], "gather_frac_of_measured_copy": g["gbs"] / peak if g["gbs"] else None,
           "gather_frac_of_nominal_8000": g["gbs"] / 8000.0 if g["gbs"] else None, "write_gbs": sc["gbs"],
           "plan_ms": phases["plan"], "phase_ms": phases, "host_tier_bytes_per_step": host_b,
           "l2": "L2 flushed between steps" if job.fits_l2() else "inputs larger than L2", "ring_model_matches": job.ring_ok}
    if job.w.host_pages:
        res["host_link_gbs"] = {k: (host_b / kern[k]["ms_per_step"] / 1e6 if kern[k]["ms_per_step"] > 0 else None) for k in ("gather_host", "scatter_host")}
    job.close()
    del job
    gc.collect()
    import torch
    torch.cuda.empty_cache()
    return res


def all_configs(args):
    """Every other configuration the benchmark spec names, one short pass each (the headline configuration is the line itself)."""
    out = {}
    for key, name, hbm in (("tiny", "tiny", True), ("video_heavy", "video_heavy", True), ("host_tier_stress", "host_tier_stress", False),
                           ("host_tier_stress_all_hbm", "host_tier_stress", True)):
        try:
            out[key] = short_pass(args, name, hbm)
        except Exception as e:   # a configuration that does not fit this box must not take the line down
            out[key] = {"error": repr(e)[:200]}
    for ps in (2 << 20, 4096):
        try:
            r = sweep_measure(args, ps, with_variants=False)
            out[f"frag_sweep_{ps}"] = {k: r[k] for k in ("value", "unit", "residents", "packed_tokens", "microbatches", "gather_ms", "gather_launches",
                                                          "frac_of_measured_peak", "frac_of_nominal_8000", "write_gbs", "plan_ms_host_wall_median",
                                                          "internal_fragmentation", "padding_waste", "rank_imbalance")}
            out[f"frag_sweep_{ps}"]["workload"] = r["config"]["workload"]
        except Exception as e:
            out[f"frag_sweep_{ps}"] = {"error": repr(e)[:200]}
    return out


def run_backbone_only(args):
    """One JSON line with the backbone-side measurements alone (small cases for profiler captures)."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    job = DeviceJob(args, True)
    res = backbone_side(job, reps=max(1, args.steps))
    job.close()
    print(json.dumps({"workload": workload_label(args) + " (all HBM)", "samples": job.w.n_samples, "backbone_side": res}))


def init_dist(torch):
    """Process group of this run (None outside torchrun): NCCL, one rank per GPU; FLOWPOOL_BENCH_BACKEND=gloo lets
    several ranks share a GPU (how the multi-rank code path is exercised where only one GPU is at hand)."""
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    backend = os.environ.get("FLOWPOOL_BENCH_BACKEND", "nccl")
    if backend != "nccl":
        local %= max(1, torch.cuda.device_count())
    torch.cuda.set_device(local)
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:   # under torchrun, also at one rank: same code path at every N
        import torch.distributed as dist
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    return dist, rank, local, world, backend


def roofline_of(kern, peak, peak_src):
    g = kern["gather_device"] if kern["gather_device"]["ms_per_step"] > 0 else kern["gather_host"]
    achieved = g["gbs"]
    per_launch = g["bytes_per_step"] / max(1.0, g["launches_per_step"])
    return {
        "kernel": "k_gather (device-tier rows)", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak if achieved else None, "peak_source": peak_src + "; a plain copy, not a hardware limit: a fraction slightly above 1 is possible",
        "algorithmic_bytes_per_launch": per_launch, "ms_per_launch": g["ms_per_step"] / max(1.0, g["launches_per_step"]),
        "traffic": per_launch * NCU_TRAFFIC_RATIO_GATHER if NCU_TRAFFIC_RATIO_GATHER else None,
        "traffic_note": "dram__bytes_read + dram__bytes_write of one launch on the first 64 samples (all HBM), scaled by the tokens "
                        "of a full launch; an upper bound at full size, where more table rows are served from L2",
        "frac_of_nominal_8000": achieved / 8000.0 if achieved else None,
    }


def run_ours(args):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the product path)")
    dist, rank, local, world, backend = init_dist(torch)
    sampler = ClockSampler(local)
    job = DeviceJob(args, args.all_hbm)
    w = job.w
    sampler.start()
    ms, prof, launches, n_mb = timed_steps(job, args.steps, args.warmup, dist)
    clocks = sampler.stop()
    wb, gb = algorithmic_bytes(w)
    value = aggregate_value(wb + gb, world, ms)
    kern, host_b = kernel_breakdown(job, prof, args.steps)
    phases = phase_breakdown(job)
    link = measure_host_link(torch) if (w.host_pages and rank == 0) else None
    if link:
        # bytes that cross the link per step: host-tier vision bytes, once per direction
        for k, ref in (("gather_host", "h2d_gbs"), ("scatter_host", "d2h_gbs")):
            ms_k = kern[k]["ms_per_step"]
            if ms_k > 0:
                kern[k]["link_gbs"] = host_b / ms_k / 1e6
                kern[k]["link_frac_of_memcpy"] = kern[k]["link_gbs"] / link[ref]

    line = None
    peak, peak_src = measured_peak()
    if rank == 0:
        hb = job.host_bytes_per_step
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic",
            "config": {"workload": workload_label(args), "samples": w.n_samples, "packed_tokens": w.total_tokens,
                       "vision_tokens": w.total_vision_tokens, "microbatches": n_mb, "hbm_pages": w.hbm_pages,
                       "host_pages": w.host_pages,
                       "bind_order": "identity" if w.bind_order == 0 else "seeded permutation", "tuning": args.tuning,
                       "host_tier_bytes_per_step": {"min": int(min(hb)), "mean": float(np.mean(hb)), "max": int(max(hb)),
                                                    "ring_model_matches_pool": job.ring_ok,
                                                    "note": "the free ring rotates from step to step (pool = 1.02 x one batch), so the bytes "
                                                            "that land on host-tier pages, and with them the link-bound step time, differ per "
                                                            "step; the kernel figures use the bytes the timed steps moved"},
                       "l2": ("L2 flushed between steps (512 MiB scrub outside the timed regions)" if job.fits_l2()
                              else "inputs larger than L2 (no flush needed)"), "parallelism": f"dp{world} (independent batches)"},
            "tokens_per_s": world * w.total_tokens / ms * 1e3,
            "gpu_launches": launches, "kernels": kern, "phase_ms": phases, "plan_call_host_ms_in_step": job.plan_ms_in_step,
            "host_link_memcpy": link, "roofline": roofline_of(kern, peak, peak_src), "clocks": clocks,
        }
    # end to end through host buffers, on the same pool as the headline number
    if rank == 0:
        if not args.skip_e2e and world == 1:
            line["e2e"] = run_e2e(job, max(1, min(args.steps, 2)))
        else:
            line["e2e"] = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                           "note": "measured at --gpus 1"}
    if rank == 0 and world == 1 and args.all_hbm and not args.skip_variants:
        line["backbone_side"] = backbone_side(job)
    # all-HBM variant of the same batch (the benchmark spec's target is stated for HBM-resident pools)
    if not args.all_hbm and not args.skip_variants:
        job.close()
        job = DeviceJob(args, True)
        ms2, prof2, _, _ = timed_steps(job, args.steps, args.warmup, dist)
        kern2, _ = kernel_breakdown(job, prof2, args.steps)
        phases2 = phase_breakdown(job)
        if rank == 0:
            g2 = kern2["gather_device"]
            line["all_hbm_variant"] = {"value": world * (wb + gb) / ms2 / 1e6, "unit": UNIT, "ms_per_step": ms2,
                                       "tokens_per_s": world * w.total_tokens / ms2 * 1e3, "kernels": kern2,
                                       "phase_ms": phases2, "plan_call_host_ms_in_step": job.plan_ms_in_step,
                                       "gather_frac_of_measured_peak": g2["gbs"] / peak if g2["gbs"] else None,
                                       "gather_frac_of_nominal_8000": g2["gbs"] / 8000.0 if g2["gbs"] else None}
            # the driver's record keeps `roofline` whole: the HBM-resident figures ride in it too
            line["roofline"]["all_hbm_pool"] = {"achieved": g2["gbs"], "frac": g2["gbs"] / peak, "frac_of_nominal_8000": g2["gbs"] / 8000.0,
                                                "ms_per_launch": g2["ms_per_step"], "algorithmic_bytes_per_launch": g2["bytes_per_step"],
                                                "whole_step_gbs": line["all_hbm_variant"]["value"], "whole_step_ms": ms2,
                                                "scatter_gbs": kern2["scatter_device"]["gbs"]}
            if world == 1:
                line["all_hbm_variant"]["backbone_side"] = backbone_side(job)
    job.close()
    del job          # its resident inputs and outputs go before the streaming measurement builds its own
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.skip_variants:
        # the decoupled producer/consumer flow on the headline pool's tier split (and all-HBM beside it)
        line["streaming"] = run_streaming(args, args.all_hbm)
        if not args.all_hbm:
            line["all_hbm_variant"]["streaming"] = run_streaming(args, True)
    if world == 1 and rank == 0 and not args.skip_variants and not args.skip_configs and args.workload == "image_mix_7b" and not args.samples:
        line["all_configs"] = all_configs(args)
        line["roofline"]["other_configs"] = {k: {kk: v.get(kk) for kk in ("gather_gbs", "gather_frac_of_measured_copy", "write_gbs", "step_ms", "value",
                                                                        "frac_of_measured_peak", "gather_ms")
                                                 if v.get(kk) is not None} for k, v in line["all_configs"].items()}
    if world > 1 and not args.skip_variants:
        # the paper's own multi-process flow: every rank writes, descriptors are exchanged, all plan alike, each
        # assembles the share Algorithm 1 dealt to it from everybody's pages
        ex = exchange_measure(args, dist, rank, world, local, backend)
        if rank == 0:
            line["exchange"] = ex
    if rank == 0:
        if world == 1 and not args.skip_cpu:
            n = min(CPU_SAMPLE, w.n_samples)
            r = time_oracle(args.workload, n, args.all_hbm, 4, 1)   # about 15 s of CPU work on this workload
            line["cpu_baseline"] = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}
            line["cpu_baseline"]["assembly_only"] = time_oracle_gather_threads(args.workload, n, args.all_hbm)
        print(json.dumps(line))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# scale + fragmentation sweep (one page size per invocation)
# ---------------------------------------------------------------------------------------------
def run_sweep(args):
    """Config 5 for one page size: prints sweep_measure's line."""
    import torch
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    args.sweep_samples = args.samples
    print(json.dumps(sweep_measure(args, args.page_bytes)))


def sweep_measure(args, PS, with_variants=True):
    """Config 5: a stream of samples flows through a fixed-capacity pool (10 x {admit while it fits, free a
    seeded half}, final admit), then the residents are planned and gathered.  Returns one line (a dict) with the
    gather/write bandwidth, plan time, fragmentation and packing figures for the given page size."""
    import torch
    import workloads
    from harness import pool_config_fields, plan_config_fields, register_args, write_args
    from paper_2606_23087_b200 import binding as fp
    st = torch.cuda.current_stream().cuda_stream
    pool_gib = args.pool_gib
    if torch.cuda.mem_get_info()[0] < (pool_gib + 26) * (1 << 30):
        pool_gib /= 2          # a box with less free memory runs the same churn through half the capacity
    w = workloads.make_workload("frag_sweep", n_samples=getattr(args, "sweep_samples", None) or 65536, page_bytes=PS,
                                pool_bytes=int(pool_gib * (1 << 30)))
    ops, residents = workloads.admit_free_schedule(w, cycles=args.cycles)
    pool = fp.Pool(fp.PoolConfig(**pool_config_fields(w)))
    if pool.rc != 0:
        raise fp.FlowpoolError(pool.rc, "pool_create")
    apply_tuning(pool, args)
    pool.profile_enable(True)
    written_vis = 0
    consumed = 0
    for kind, samples in ops:
        if kind == "free":
            rc = pool.free(samples, st)
            assert rc == 0, rc
            continue
        consumed += len(samples)
        for i in range(0, len(samples), 256):
            part = samples[i:i + 256]
            reg = register_args(w, part)
            ids = torch.from_numpy(reg[5]).cuda()
            srcs = [workloads.span_values(w, s, 0, device="cuda") for s in part]
            assert pool.register_samples(*reg[:5], ids.data_ptr(), st) == 0
            rc = pool.write_embeddings(*write_args(w, [(s, 0) for s in part]), [t.data_ptr() for t in srcs], 0, st)
            assert rc == 0, rc
            torch.cuda.synchronize()
            written_vis += int(sum(int(w.spans_of(s)[1][0]) for s in part))
    prof_w = pool.profile_read()
    write_ms = prof_w["scatter_device"]["ms"]
    stats = pool.stats()
    # plan the residents (admission order)
    order = np.asarray(residents, dtype=np.uint32)
    pcfg = fp.PlanConfig(**plan_config_fields(w))
    plan_ms = []
    plan = None
    for _ in range(3):
        if plan:
            plan.destroy()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        rc, plan = pool.plan_microbatches(order, pcfg, st)
        plan_ms.append((time.perf_counter() - t0) * 1e3)
        assert rc == 0, rc
    a = plan.arrays()
    n_mb, total_tokens, _ = plan.summary()
    # scheduler variants on the same residents: what each buys in padding waste and rank balance
    variants = {}
    for name, fl, k_limit in ((("default", 0, 0), ("longest_first", 2, 0), ("sum_of_squares", 4, 0), ("carried_zigzag", 8, 0),
                               ("all_three", 14, 0), ("auto_k_limit_64", 16, 64), ("fixed_k_64", 0, 64)) if with_variants else ()):
        vc = plan_config_fields(w, flags=fl)
        if k_limit:
            vc["n_buckets_K"] = k_limit
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        rc, vp = pool.plan_microbatches(order, fp.PlanConfig(**vc), st)
        dt = (time.perf_counter() - t0) * 1e3
        assert rc == 0, rc
        va = vp.arrays()
        vl = np.array([va["mb_cost"][va["mb_rank"] == r].astype(np.float64).sum() for r in range(w.n_ranks_N)])
        variants[name] = {"microbatches": int(va["n_mb"]), "padding_waste": 1.0 - total_tokens / (int(va["n_mb"]) * w.budget_L),
                          "rank_imbalance": float((vl.max() - vl.min()) / vl.mean()), "plan_ms_host_wall": dt,
                          "buckets_used": int(len(np.unique(va["mb_bucket"])))}
        vp.destroy()
    # gather everything, in ranges that fit a reusable output buffer
    table = workloads.embed_table(w, device="cuda")
    buf_rows = min(total_tokens, 1 << 20)
    out = torch.empty((buf_rows, w.hidden), dtype=torch.bfloat16, device="cuda")
    cu = torch.empty((len(residents) + n_mb + 8,), dtype=torch.int32, device="cuda")
    pos = torch.empty((buf_rows,), dtype=torch.int32, device="cuda")
    ranges, b, rows = [], 0, 0
    for j in range(n_mb):
        t = int(a["mb_tokens"][j])
        if rows + t > buf_rows:
            ranges.append((b, j)); b, rows = j, 0
        rows += t
    ranges.append((b, n_mb))
    gather_ms = None
    for rep in range(3):
        pool.profile_read()
        for lo, hi in ranges:
            rc = pool.gather_packed(plan, lo, hi, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), st)
            assert rc == 0, rc
        g = pool.profile_read()["gather_device"]
        gather_ms = g["ms"] if gather_ms is None else min(gather_ms, g["ms"])
    assert pool.status() == (0, 0)
    # planner scale: every descriptor of the stream, metadata only (needs free slots: use a second pool)
    plan.destroy()
    # fragmentation figures
    need_bytes = sum(int(w.spans_of(s)[1][0]) * w.row_bytes for s in residents)
    used_pages = stats["pages_total"] - stats["pages_free"]
    runs = []
    for s in residents[:: max(1, len(residents) // 200)]:
        pg = pool.span_pages(s, 0, cap=1 << 16)[1].astype(np.int64)
        if len(pg) > 1:
            brk = int((np.diff(pg) != PS).sum())
            runs.append(len(pg) / (brk + 1))
        elif len(pg) == 1:
            runs.append(1.0)
    loads = np.array([a["mb_cost"][a["mb_rank"] == r].astype(np.float64).sum() for r in range(w.n_ranks_N)])
    row_b = w.row_bytes
    peak, peak_src = measured_peak()
    gbs = 2 * total_tokens * row_b / gather_ms / 1e6
    line = {
        "metric": "packed-microbatch assembly GB/s after churn (fragmentation sweep)", "value": gbs, "unit": "GB/s",
        "n_gpus": 1, "higher_is_better": True, "dtype": "u8", "data": "synthetic",
        "config": {"workload": f"frag_sweep: stream of {w.n_samples} samples, hidden {w.hidden}, page {PS} B, pool "
                               f"{pool_gib} GiB all HBM, {args.cycles} write/free cycles, budget {w.budget_L}",
                   "page_bytes": PS},
        "residents": len(residents), "stream_consumed": consumed, "packed_tokens": int(total_tokens), "microbatches": n_mb,
        "gather_ms": gather_ms, "gather_launches": len(ranges), "frac_of_measured_peak": gbs / peak, "frac_of_nominal_8000": gbs / 8000.0,
        "write_gbs": 2 * written_vis * row_b / write_ms / 1e6, "write_ms_total": write_ms,
        "plan_ms_host_wall_median": float(np.median(plan_ms)),
        "internal_fragmentation": 1.0 - need_bytes / (used_pages * PS),
        "mean_contiguous_run_pages": float(np.mean(runs)) if runs else None,
        "padding_waste": 1.0 - total_tokens / (n_mb * w.budget_L),
        "rank_imbalance": float((loads.max() - loads.min()) / loads.mean()),
        "plan_variants": variants,
        "gpu_launches": pool.stats()["gpu_launches"],
    }
    pool.destroy()
    del out, table
    torch.cuda.empty_cache()
    return line


# ---------------------------------------------------------------------------------------------
# streaming: producer stream and consumer stream overlap successive batches
# ---------------------------------------------------------------------------------------------
def run_streaming(args, all_hbm, batches=6, warm=2):
    """The decoupled flow (Sec. 3.1): while the consumer stream plans and assembles batch k, the producer stream
    registers and writes batch k+1 into a pool that holds two batches; pool_free recycles batch k on the producer
    stream as soon as it is assembled.  Returns steady-state ms per batch and the whole-path GB/s."""
    import torch
    import workloads
    from harness import pool_config_fields, plan_config_fields, register_args, write_args
    from paper_2606_23087_b200 import binding as fp
    w = workloads.make_workload(args.workload, n_samples=args.samples, all_hbm=all_hbm, id_skew=getattr(args, "id_skew", "uniform"))
    n = w.n_samples
    f = pool_config_fields(w, max_samples=2 * n)
    f["hbm_pages"], f["host_pages"] = 2 * w.hbm_pages, 2 * w.host_pages
    f["max_text_tokens"] = 2 * w.total_text_tokens_capacity
    # pages of both tiers interleaved in the free ring: every batch then carries its share of host-tier pages, and
    # the host-tier writes of batch k+1 (device -> host) can overlap the host-tier reads of batch k (host -> device)
    f["ring_order"] = 1
    pool = fp.Pool(fp.PoolConfig(**f))
    if pool.rc != 0:
        raise fp.FlowpoolError(pool.rc, "pool_create")
    apply_tuning(pool, args)
    prod, cons = torch.cuda.Stream(), torch.cuda.Stream()
    table = workloads.embed_table(w, device="cuda")
    calls = []
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        reg = register_args(w, samples)
        wr = write_args(w, call)
        srcs = [workloads.span_values(w, s, j, device="cuda") for s, j in call]
        calls.append((reg, torch.from_numpy(reg[5]).cuda(), wr, [t.data_ptr() for t in srcs], srcs))
    outs = [torch.empty((w.total_tokens, w.hidden), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    cu = torch.empty((2 * n + 8,), dtype=torch.int32, device="cuda")
    pos = torch.empty((w.total_tokens,), dtype=torch.int32, device="cuda")
    pcfg = fp.PlanConfig(**plan_config_fields(w))

    def produce(k):
        off = (k % 2) * n
        for reg, ids, wr, ptrs, _ in calls:
            rc = pool.register_samples(reg[0] + off, *reg[1:5], ids.data_ptr(), prod.cuda_stream)
            assert rc == 0, rc
            rc = pool.write_embeddings(wr[0] + off, wr[1], wr[2], ptrs, w.src_dtype, prod.cuda_stream)
            assert rc == 0, rc

    def make_plan():
        rc, slots, _ = pool.take_ready(w.total_tokens, n)      # watermark: one whole batch is ready
        assert rc == 0 and len(slots) == n, (rc, len(slots))
        rc, plan = pool.plan_microbatches(slots, pcfg, cons.cuda_stream)
        assert rc == 0, rc
        return slots, plan

    def assemble(k, plan):
        n_mb = plan.summary()[0]
        rc = pool.gather_packed(plan, 0, n_mb, table.data_ptr(), w.vocab, outs[k % 2].data_ptr(), cu.data_ptr(), pos.data_ptr(),
                                cons.cuda_stream)
        assert rc == 0, rc

    # Issue order per round: assemble batch k (consumer stream); write batch k+1 (producer stream); plan batch k+1 as
    # soon as its write calls are queued (the plan needs the metadata only, which the metadata stream has ready long
    # before the copies end); free batch k (the library makes it wait for the assembly).  The consumer waits only for
    # producer calls issued before it, so the write of k+1 and the assembly of k run side by side, and no round
    # starts by waiting for a plan.
    torch.cuda.synchronize()
    produce(0)
    slots, plan = make_plan()
    t0 = None
    total = warm + batches
    for k in range(total):
        if k == warm:
            torch.cuda.synchronize()
            pool.profile_read()
            pool.profile_enable(True)
            t0 = time.perf_counter()
        assemble(k, plan)
        produce(k + 1)
        next_slots, next_plan = make_plan()
        assert pool.free(slots, prod.cuda_stream) == 0
        plan.destroy()
        slots, plan = next_slots, next_plan
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3 / batches
    prof = pool.profile_read()
    pool.profile_enable(False)
    kernel_ms = {k: v["ms"] / batches for k, v in prof.items() if v["launches"]}
    # drain the batch that was produced and planned but never consumed
    plan.destroy()
    pool.free(slots, prod.cuda_stream)
    assert pool.status() == (0, 0)
    wb, gb = algorithmic_bytes(w)
    pool.destroy()
    del calls, outs, table
    torch.cuda.empty_cache()
    return {"ms_per_batch": ms, "value": (wb + gb) / ms / 1e6, "unit": UNIT, "tokens_per_s": w.total_tokens / ms * 1e3,
            "batches": batches, "kernel_ms_per_batch": kernel_ms,
            "pool": "two batches resident, same tier split, tiers interleaved in the free ring",
            "note": "host wall clock over steady-state batches; producer and consumer on two streams"}


# ---------------------------------------------------------------------------------------------
# two processes of one GVA space, emulated on one GPU: producer pool (rank 1) -> consumer pool (rank 0)
# ---------------------------------------------------------------------------------------------
def _peer_producer_process(args_dict, to_parent, from_parent):
    """The producer of --via-peer --two-processes: owns rank 1's pool in a process of its own."""
    import torch
    import workloads
    from harness import pool_config_fields, register_args, write_args
    from paper_2606_23087_b200 import binding as fp
    try:
        torch.cuda.set_device(0)
        st = torch.cuda.current_stream().cuda_stream
        w = workloads.make_workload(args_dict["workload"], n_samples=args_dict["samples"], all_hbm=True)
        f = pool_config_fields(w, max_samples=w.n_samples)
        f.update(world_size=2, rank=1)
        prod = fp.Pool(fp.PoolConfig(**f))
        assert prod.rc == 0
        calls = []
        for call in w.write_calls:
            samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
            reg = register_args(w, samples)
            calls.append((reg[:5], torch.from_numpy(reg[5]).cuda(), write_args(w, call),
                          [workloads.span_values(w, s, j, device="cuda") for s, j in call]))
        order = np.asarray(w.plan_order, dtype=np.uint32)
        rc, mblob = prod.export_mapping()
        rc2, handles = prod.ipc_export()
        assert rc == 0 and rc2 == 0
        to_parent.put(("mapping", mblob.tobytes(), handles))
        while True:
            cmd = from_parent.get(timeout=600)
            if cmd == "write":
                for reg, ids, wr, srcs in calls:
                    assert prod.register_samples(*reg, ids.data_ptr(), st) == 0
                    assert prod.write_embeddings(*wr, [t.data_ptr() for t in srcs], w.src_dtype, st) == 0
                rc, sblob = prod.export_samples(order, st)    # synchronises the stream: the pages are written
                assert rc == 0
                to_parent.put(("samples", sblob.tobytes()))
            elif cmd == "free":
                assert prod.free(order, st) == 0
                torch.cuda.synchronize()
                to_parent.put(("freed",))
            else:
                break
        assert prod.status() == (0, 0)
        prod.destroy()
        to_parent.put(("bye",))
    except BaseException as e:
        to_parent.put(("error", repr(e)))
        raise


def run_peer_two_processes(args):
    """--via-peer with the producer in a process of its own: its slabs reach the consumer through CUDA IPC handles,
    its mapping and its samples' descriptors through a host queue.  All pages in HBM (host-tier slabs are not shared
    by these calls).  One GPU: the two processes' segments are in the same HBM."""
    import multiprocessing as mp
    import torch
    import workloads
    from harness import pool_config_fields, plan_config_fields
    from paper_2606_23087_b200 import binding as fp
    torch.cuda.set_device(0)
    st = torch.cuda.current_stream().cuda_stream
    w = workloads.make_workload(args.workload, n_samples=args.samples, all_hbm=True)
    n = w.n_samples
    ctx = mp.get_context("spawn")
    to_child, from_child = ctx.Queue(), ctx.Queue()
    child = ctx.Process(target=_peer_producer_process, args=({"workload": args.workload, "samples": args.samples}, from_child, to_child),
                        daemon=True)
    child.start()
    try:
        f = pool_config_fields(w, max_samples=n)
        f.update(world_size=2, rank=0, hbm_pages=64, host_pages=0, max_imported_pages=w.hbm_pages + w.host_pages)
        cons = fp.Pool(fp.PoolConfig(**f))
        assert cons.rc == 0
        msg = from_child.get(timeout=600)
        assert msg[0] == "mapping", msg
        rc, hbm, text = fp.ipc_open(msg[2])
        assert rc == 0 and cons.import_mapping(np.frombuffer(msg[1], np.uint8), hbm, 0, text) == 0
        table = workloads.embed_table(w, device="cuda")
        out = torch.empty((w.total_tokens, w.hidden), dtype=torch.bfloat16, device="cuda")
        cu = torch.empty((2 * n + 8,), dtype=torch.int32, device="cuda")
        pos = torch.empty((w.total_tokens,), dtype=torch.int32, device="cuda")
        order = np.asarray(w.plan_order, dtype=np.uint32)
        pcfg = fp.PlanConfig(**plan_config_fields(w))
        cons.profile_enable(True)
        n_mb, blob_bytes, xfer_ms = 0, 0, []
        for it in range(args.warmup + args.steps):
            to_child.put("write")
            msg = from_child.get(timeout=600)
            assert msg[0] == "samples", msg
            t0 = time.perf_counter()
            sblob = np.frombuffer(msg[1], np.uint8)
            assert cons.import_samples(order, sblob, st) == 0
            torch.cuda.synchronize()
            xfer_ms.append((time.perf_counter() - t0) * 1e3)
            rc, plan = cons.plan_microbatches(order, pcfg, st)
            assert rc == 0
            n_mb = plan.summary()[0]
            if it == args.warmup:
                cons.profile_read()
            assert cons.gather_packed(plan, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), st) == 0
            assert cons.free(order, st) == 0
            plan.destroy()
            torch.cuda.synchronize()
            to_child.put("free")
            assert from_child.get(timeout=600)[0] == "freed"
            blob_bytes = len(sblob)
        prof = cons.profile_read()
        assert cons.status() == (0, 0)
        # spot-check a few rows against the generator: text rows of the first sample
        ids0 = workloads.input_ids(w, int(order[0]))
        row = int(np.nonzero(ids0 != w.placeholder_id)[0][0])
        ok = bool(torch.equal(out[row], table[int(ids0[row])]))
        cons.destroy()
        assert fp.ipc_close(hbm, text) == 0
        to_child.put("quit")
        assert from_child.get(timeout=600)[0] == "bye"
        child.join(timeout=60)
    finally:
        if child.is_alive():
            child.kill()   # this very process object
    g_ms = prof["gather_device"]["ms"] / args.steps
    peak, _ = measured_peak()
    gbs = 2 * w.total_tokens * w.row_bytes / g_ms / 1e6
    args.all_hbm = True
    label = workload_label(args)
    print(json.dumps({"metric": "packed-microbatch assembly GB/s, consumer process reading a producer process's pages (CUDA IPC, one GPU)",
                      "value": gbs, "unit": "GB/s", "n_gpus": 1, "higher_is_better": True, "dtype": "u8", "data": "synthetic",
                      "config": {"workload": label, "processes": 2, "note": "both segments in the same HBM"},
                      "gather_device_ms": g_ms, "frac_of_measured_peak": gbs / peak, "descriptor_import_ms": float(np.median(xfer_ms[args.warmup:])),
                      "descriptor_blob_bytes": blob_bytes, "microbatches": n_mb, "sampled_row_matches": ok}))


class BlobExchange:
    """Every rank's variable-length byte blob to every rank in one all_gather_into_tensor over preallocated,
    length-prefixed fixed-size slots (no pickling on the per-step path)."""

    def __init__(self, dist, cap, device):
        import torch
        self.dist, self.cap, self.world = dist, int(cap), dist.get_world_size()
        self.send = torch.zeros(self.cap + 8, dtype=torch.uint8, device=device)
        self.recv = torch.zeros(self.world * (self.cap + 8), dtype=torch.uint8, device=device)
        self.stage = torch.zeros(self.cap + 8, dtype=torch.uint8, pin_memory=(device != "cpu"))

    @staticmethod
    def agree_cap(dist, nbytes, device):
        """The largest blob over all ranks (one all_reduce, at set-up)."""
        import torch
        t = torch.tensor([int(nbytes)], dtype=torch.int64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return int(t.item())

    def all_gather(self, blob):
        blob = np.ascontiguousarray(blob, dtype=np.uint8)
        n = len(blob)
        if n > self.cap:
            raise ValueError(f"blob of {n} bytes exceeds the exchange slot of {self.cap}")
        st = self.stage.numpy()
        st[:8] = np.frombuffer(np.uint64(n).tobytes(), dtype=np.uint8)
        st[8:8 + n] = blob
        self.send.copy_(self.stage)
        self.dist.all_gather_into_tensor(self.recv, self.send)
        r = self.recv.cpu().numpy().reshape(self.world, self.cap + 8)
        return [r[i, 8:8 + int(r[i, :8].copy().view(np.uint64)[0])].copy() for i in range(self.world)]


def exchange_measure(args, dist, rank, world, local, backend):
    """The paper's own setting (Sec. 3.2, 3.4) with one process per rank: every rank writes its batch into its own
    segment; mappings and slab handles are exchanged once, the samples' descriptors every step; every rank plans ALL
    samples (Algorithm 1 is deterministic, so the plans agree) and assembles only the microbatches dealt to it,
    reading the other ranks' pages in place (peer loads over NVLink when the ranks own different GPUs).  All pages
    in HBM.  Returns rank 0's summary (None elsewhere)."""
    import torch
    import workloads
    from harness import pool_config_fields, plan_config_fields, register_args, write_args
    from paper_2606_23087_b200 import binding as fp
    dev = "cuda" if backend == "nccl" else "cpu"
    st = torch.cuda.current_stream().cuda_stream
    w = workloads.make_workload(args.workload, n_samples=args.samples, all_hbm=True)
    n = w.n_samples
    f = pool_config_fields(w, max_samples=world * n)
    f.update(world_size=world, rank=rank, bind_seed=100 + rank, ring_seed=200 + rank,
             max_imported_pages=(world - 1) * (w.hbm_pages + w.host_pages), max_text_tokens=world * w.total_text_tokens_capacity)
    pool = fp.Pool(fp.PoolConfig(**f))
    assert pool.rc == 0, pool.rc
    apply_tuning(pool, args)
    # once: everybody's mapping and slab handles
    rc1, mblob = pool.export_mapping()
    rc2, handles = pool.ipc_export()
    assert rc1 == 0 and rc2 == 0
    init_blob = np.concatenate([np.frombuffer(handles, np.uint8), mblob])
    everyone = BlobExchange(dist, BlobExchange.agree_cap(dist, len(init_blob), dev), dev).all_gather(init_blob)
    opened = []
    for r, blob in enumerate(everyone):
        if r == rank:
            continue
        rc, hbm, text = fp.ipc_open(blob[:fp.IPC_HANDLES_BYTES].tobytes())
        assert rc == 0, rc
        opened.append((hbm, text))
        assert pool.import_mapping(blob[fp.IPC_HANDLES_BYTES:], hbm, 0, text) == 0
    # own batch: global sample g = rank * n + s lives in slot g on every rank
    calls = []
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        reg = register_args(w, samples)
        slots = (np.asarray(reg[0], np.uint32) + rank * n).astype(np.uint32)
        wr = write_args(w, call)
        calls.append(((slots,) + tuple(reg[1:5]), torch.from_numpy(reg[5]).cuda(),
                      ((np.asarray(wr[0], np.uint32) + rank * n).astype(np.uint32),) + tuple(wr[1:]),
                      [workloads.span_values(w, s, j, device="cuda") for s, j in call]))
    plan_order = np.asarray(w.plan_order, np.uint32)
    own = (plan_order + rank * n).astype(np.uint32)
    order = np.concatenate([(plan_order + r * n) for r in range(world)]).astype(np.uint32)
    pc = plan_config_fields(w)
    pc["n_ranks_N"] = world
    pcfg = fp.PlanConfig(**pc)
    table = workloads.embed_table(w, device="cuda")
    cap_rows = int(w.total_tokens * 1.5) + w.budget_L
    out = torch.empty((cap_rows, w.hidden), dtype=torch.bfloat16, device="cuda")
    cu = torch.empty((2 * world * n + 8,), dtype=torch.int32, device="cuda")
    pos = torch.empty((cap_rows,), dtype=torch.int32, device="cuda")
    vis_of = np.array([int(w.spans_of(s)[1].astype(np.int64).sum()) for s in range(n)], dtype=np.int64)
    step_ms, my_rows, n_mb, remote_b, xchg = [], 0, 0, 0, None
    pool.profile_enable(True)
    sampler = ClockSampler(local)
    for it in range(args.warmup + args.steps):
        if it == args.warmup:
            pool.profile_read()
            if rank == 0:
                sampler.start()
        dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for reg, ids, wr, srcs in calls:
            assert pool.register_samples(*reg, ids.data_ptr(), st) == 0
            assert pool.write_embeddings(*wr, [t.data_ptr() for t in srcs], w.src_dtype, st) == 0
        rc, sblob = pool.export_samples(own, st)          # returns with this rank's pages written
        assert rc == 0
        if xchg is None:                                  # first (warm-up) step: agree on the slot size, allocate once
            xchg = BlobExchange(dist, BlobExchange.agree_cap(dist, len(sblob), dev), dev)
        blobs = xchg.all_gather(sblob)                    # the per-round exchange of "lightweight metadata"
        for r in range(world):
            if r != rank:
                assert pool.import_samples((plan_order + r * n).astype(np.uint32), blobs[r], st) == 0
        rc, plan = pool.plan_microbatches(order, pcfg, st)
        assert rc == 0
        pa = plan.arrays()
        n_mb = int(pa["n_mb"])
        mine = [int(j) for j in pa["rank_mbs"][pa["rank_mb_off"][rank]:pa["rank_mb_off"][rank + 1]]]
        my_rows = int(pa["mb_tokens"][mine].sum()) if mine else 0
        assert my_rows <= cap_rows
        if mine:
            assert pool.gather_list(plan, mine, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), st) == 0
        e1.record()
        torch.cuda.synchronize()
        # bytes this rank read from other ranks' memory: vision rows and token ids of the samples it assembled but does not own
        remote_b = 0
        for j in mine:
            for g in pa["mb_samples"][pa["mb_sample_off"][j]:pa["mb_sample_off"][j + 1]]:
                g = int(g)
                if g // n != rank:
                    remote_b += int(vis_of[g % n]) * w.row_bytes + 4 * int(w.seq_len[g % n])
        if mine and it == 0:
            # spot check against the generator: first and last row of the first sample of this rank's share
            q0 = int(pa["mb_sample_off"][mine[0]])
            g = int(pa["mb_samples"][q0])
            s_local = g % n                                  # every rank generated the same workload
            ids_s = workloads.input_ids(w, s_local)
            sp_pos, sp_tok = w.spans_of(s_local)
            for p_ in (0, len(ids_s) - 1):
                in_span = [j for j in range(len(sp_pos)) if int(sp_pos[j]) <= p_ < int(sp_pos[j]) + int(sp_tok[j])]
                if in_span:
                    j = in_span[0]
                    want = workloads.span_values(w, s_local, j, device="cuda", rows=(p_ - int(sp_pos[j]), p_ - int(sp_pos[j]) + 1))[0]
                else:
                    want = table[int(ids_s[p_])]
                assert torch.equal(out[p_].view(torch.int16), want.to(torch.bfloat16).view(torch.int16)), (rank, g, p_)
        for r in range(world):
            if r != rank:
                assert pool.free((plan_order + r * n).astype(np.uint32), st) == 0
        plan.destroy()
        torch.cuda.synchronize()
        dist.barrier()                                    # nobody reads this rank's pages any more
        assert pool.free(own, st) == 0
        torch.cuda.synchronize()
        if it >= args.warmup:
            step_ms.append(e0.elapsed_time(e1))
    clocks = sampler.stop() if rank == 0 else None
    prof = pool.profile_read()
    assert pool.status() == (0, 0)
    ms = float(np.median(step_ms))
    g_ms = prof["gather_device"]["ms"] / max(1, args.steps)
    t = torch.tensor([ms, float(my_rows), g_ms, float(remote_b)], dtype=torch.float64, device=dev)
    allv = [torch.zeros_like(t) for _ in range(world)]
    dist.all_gather(allv, t)
    per = np.array([v.cpu().numpy() for v in allv])
    ms_max, rows_all = float(per[:, 0].max()), float(per[:, 1].sum())
    wb, _ = algorithmic_bytes(w)
    moved = world * wb + rows_all * 4 * w.hidden
    pool.destroy()
    for hbm, text in opened:
        fp.ipc_close(hbm, text)
    if rank != 0:
        return None
    peak, peak_src = measured_peak()
    nvlink_gbs = 770.0      # measured peer copy per direction on this machine
    n_dev = min(world, torch.cuda.device_count())
    per_rank = []
    for r in range(world):
        rows_r, gms_r, rem_r = float(per[r, 1]), float(per[r, 2]), float(per[r, 3])
        gb_r = rows_r * 4 * w.hidden
        # rows read from a peer GPU cannot come faster than the link; ranks that share one GPU share its HBM instead
        bound_ms = max(gb_r / peak, rem_r / nvlink_gbs if n_dev > 1 else 0.0) / 1e6
        per_rank.append({"rank": r, "rows": int(rows_r), "gather_ms": gms_r, "gather_gbs": gb_r / gms_r / 1e6 if gms_r > 0 else None,
                         "bytes_from_peers": int(rem_r), "roofline_bound_ms": bound_ms, "frac_of_bound": bound_ms / gms_r if gms_r > 0 else None})
    slow = max(per_rank, key=lambda x: x["gather_ms"])
    return {"metric": METRIC + ", ranks exchanging descriptors and reading each other's pages in place", "value": moved / ms_max / 1e6,
            "unit": UNIT, "ms_per_step": ms_max, "tokens_per_s": rows_all / ms_max * 1e3,
            "config": {"workload": workload_label(args, all_hbm=True), "ranks": world, "gpus_used": n_dev, "backend": backend, "microbatches": n_mb,
                       "packed_tokens_all_ranks": int(rows_all), "pool": "all pages in HBM (host-tier slabs are not shared between processes)",
                       "exchange": "descriptors per step by all_gather_into_tensor over preallocated length-prefixed slots; host time included"},
            "per_rank": per_rank,
            "bytes_over_nvlink_per_step": int(per[:, 3].sum()) if n_dev > 1 else 0,
            "bytes_from_peer_processes_per_step": int(per[:, 3].sum()),
            "roofline": {"kernel": "k_gather (list layout), slowest rank", "bound": "hbm" if slow["roofline_bound_ms"] * 1e6 * peak >= slow["rows"] * 4 * w.hidden * 0.999 else "nvlink",
                         "achieved": slow["gather_gbs"], "peak": peak, "unit": "GB/s", "frac": slow["frac_of_bound"],
                         "peak_source": peak_src + "; peer rows bounded by 770 GB/s per direction (measured peer copy)"},
            "clocks": clocks}


def run_exchange(args):
    """--exchange: the multi-rank flow alone (under torchrun), one JSON line."""
    import torch
    dist, rank, local, world, backend = init_dist(torch)
    assert dist is not None, "--exchange needs torchrun (or --gpus N, which launches it)"
    ex = exchange_measure(args, dist, rank, world, local, backend)
    if rank == 0:
        ex.update({"n_gpus": world, "steps": args.steps, "warmup": args.warmup, "higher_is_better": True, "scaling": "weak",
                   "vs_baseline": None, "dtype": "u8", "data": "synthetic"})
        print(json.dumps(ex))
    dist.barrier()
    dist.destroy_process_group()


def run_peer(args):
    """The producer writes the batch into its own segment; the consumer imports its mapping (once) and, per step,
    the samples' descriptors, plans, and assembles every microbatch by reading the producer's pages in place.
    With one GPU both segments live in the same HBM, so this measures the path's own overheads (descriptor
    exchange, translation through imported tables), not a link."""
    import torch
    import workloads
    from harness import pool_config_fields, plan_config_fields, register_args, write_args
    from paper_2606_23087_b200 import binding as fp
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    st = torch.cuda.current_stream().cuda_stream
    w = workloads.make_workload(args.workload, n_samples=args.samples, all_hbm=args.all_hbm)
    n = w.n_samples

    def cfg(rank):
        f = pool_config_fields(w, max_samples=n)
        f.update(world_size=2, rank=rank)
        if rank == 0:  # the consumer holds no embeddings of its own here
            f.update(hbm_pages=64, host_pages=0, max_imported_pages=w.hbm_pages + w.host_pages)
        return f
    prod, cons = fp.Pool(fp.PoolConfig(**cfg(1))), fp.Pool(fp.PoolConfig(**cfg(0)))
    assert prod.rc == 0 and cons.rc == 0
    rc, mblob = prod.export_mapping()
    assert rc == 0 and cons.import_mapping(mblob, *prod.backing()) == 0
    calls = []
    for call in w.write_calls:
        samples = sorted({s for s, _ in call}, key=[s for s, _ in call].index)
        reg = register_args(w, samples)
        calls.append((reg[:5], torch.from_numpy(reg[5]).cuda(), write_args(w, call),
                      [workloads.span_values(w, s, j, device="cuda") for s, j in call]))
    table = workloads.embed_table(w, device="cuda")
    out = torch.empty((w.total_tokens, w.hidden), dtype=torch.bfloat16, device="cuda")
    cu = torch.empty((2 * n + 8,), dtype=torch.int32, device="cuda")
    pos = torch.empty((w.total_tokens,), dtype=torch.int32, device="cuda")
    order = np.asarray(w.plan_order, dtype=np.uint32)
    pcfg = fp.PlanConfig(**plan_config_fields(w))
    cons.profile_enable(True)
    xfer_ms, step_ms, blob_bytes = [], [], 0
    for it in range(args.warmup + args.steps):
        torch.cuda.synchronize()
        t_step = time.perf_counter()
        for reg, ids, wr, srcs in calls:
            assert prod.register_samples(*reg, ids.data_ptr(), st) == 0
            assert prod.write_embeddings(*wr, [t.data_ptr() for t in srcs], w.src_dtype, st) == 0
        t0 = time.perf_counter()
        rc, sblob = prod.export_samples(order, st)
        assert rc == 0 and cons.import_samples(order, sblob, st) == 0
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) * 1e3
        rc, plan = cons.plan_microbatches(order, pcfg, st)
        assert rc == 0
        n_mb = plan.summary()[0]
        if it == args.warmup:
            cons.profile_read()
        assert cons.gather_packed(plan, 0, n_mb, table.data_ptr(), w.vocab, out.data_ptr(), cu.data_ptr(), pos.data_ptr(), st) == 0
        assert cons.free(order, st) == 0 and prod.free(order, st) == 0
        plan.destroy()
        torch.cuda.synchronize()
        if it >= args.warmup:
            xfer_ms.append(dt); step_ms.append((time.perf_counter() - t_step) * 1e3); blob_bytes = len(sblob)
    prof = cons.profile_read()
    assert cons.status() == (0, 0)
    g_ms = (prof["gather_device"]["ms"] + 0.0) / args.steps
    gh_ms = prof["gather_host"]["ms"] / args.steps
    peak, _ = measured_peak()
    gbs = 2 * w.total_tokens * w.row_bytes / max(g_ms, gh_ms) / 1e6
    line = {"metric": "packed-microbatch assembly GB/s, consumer reading a peer process's pages (one GPU, emulated)",
            "value": gbs, "unit": "GB/s", "n_gpus": 1, "higher_is_better": True, "dtype": "u8", "data": "synthetic",
            "config": {"workload": workload_label(args), "ranks": 2, "note": "both segments in the same HBM"},
            "gather_device_ms": g_ms, "gather_host_ms": gh_ms, "frac_of_measured_peak": gbs / peak,
            "descriptor_export_import_ms": float(np.median(xfer_ms)), "descriptor_blob_bytes": blob_bytes,
            "step_ms_host_wall": float(np.median(step_ms)), "microbatches": n_mb}
    prod.destroy(); cons.destroy()
    print(json.dumps(line))


def self_launch(args):
    """--gpus N means N ranks.  Outside torchrun (no WORLD_SIZE in the environment) this process re-executes itself
    under `python -m torch.distributed.run` with N ranks on this node and passes their exit code on; under torchrun
    the world size must be the N asked for.  The reference arm needs no ranks: rank 0 alone runs it."""
    if args.impl == "reference":
        return
    ws = os.environ.get("WORLD_SIZE")
    if ws is not None:
        if int(ws) != args.gpus:
            raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={ws}: launch with --nproc-per-node {args.gpus}")
        return
    if args.gpus <= 1:
        return
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def run_host_logic_only(args):
    """The multi-rank plumbing of this script without a GPU (gloo on CPU): process group, slot-size agreement, the
    length-prefixed descriptor all-gather with blobs of different lengths, max-over-ranks timing, rank-0-only line."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    dist.init_process_group("gloo")
    blob = np.arange(100 + 37 * rank, dtype=np.uint64).view(np.uint8) ^ np.uint8(rank)
    xchg = BlobExchange(dist, BlobExchange.agree_cap(dist, len(blob), "cpu"), "cpu")
    ok = True
    for _ in range(2):
        got = xchg.all_gather(blob)
        for r in range(world):
            want = np.arange(100 + 37 * r, dtype=np.uint64).view(np.uint8) ^ np.uint8(r)
            ok = ok and len(got[r]) == len(want) and bool(np.array_equal(got[r], want))
    ms = max_over_ranks(10.0 + rank, dist, device="cpu")
    if rank == 0:
        print(json.dumps({"host_logic_only": True, "n_gpus": world, "blobs_ok": ok, "ms_per_step": ms,
                          "value": aggregate_value(1e6, world, ms), "unit": UNIT}))
    dist.barrier()
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="image_mix_7b")
    ap.add_argument("--all-hbm", action="store_true", help="bind every page in HBM (no host tier)")
    ap.add_argument("--samples", type=int, default=None, help="use only the first S samples (smaller case)")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-variants", action="store_true")
    ap.add_argument("--page-bytes", type=int, default=2 << 20, help="frag_sweep: page size")
    ap.add_argument("--pool-gib", type=float, default=64.0, help="frag_sweep: pool capacity")
    ap.add_argument("--cycles", type=int, default=10, help="frag_sweep: write/free cycles")
    ap.add_argument("--tuning", default=None, help="library launch-geometry knobs, e.g. dev_ctas_per_sm=4,host_ctas=6")
    ap.add_argument("--id-skew", default="uniform", choices=["uniform", "zipf"], help="distribution of the text-token ids")
    ap.add_argument("--bind-order", default="workload", choices=["workload", "identity"],
                    help="vpn -> frame binding of the main pool: the workload's (a seeded permutation) or the identity")
    ap.add_argument("--backbone-only", action="store_true", help="only the backbone-side outputs (padded assembly, table gradient) on an all-HBM pool")
    ap.add_argument("--exchange", action="store_true", help="under torchrun: every rank writes its batch, all plan everything, each assembles its own share from everybody's pages")
    ap.add_argument("--two-processes", action="store_true", help="with --via-peer: the producer pool lives in a process of its own (CUDA IPC)")
    ap.add_argument("--via-peer", action="store_true", help="producer and consumer are two processes' pools of one GVA space")
    ap.add_argument("--streaming-only", action="store_true", help="only the two-stream producer/consumer measurement")
    ap.add_argument("--skip-configs", action="store_true", help="skip the short passes over the other configurations")
    ap.add_argument("--host-logic-only", action="store_true",
                    help="no GPU work: rendezvous, the descriptor exchange and the rank-0 line only (checks of this script on CPU)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    self_launch(args)
    if args.host_logic_only:
        run_host_logic_only(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.workload == "frag_sweep":
        run_sweep(args)
    elif args.backbone_only:
        run_backbone_only(args)
    elif args.streaming_only:
        import torch
        torch.cuda.set_device(0)
        print(json.dumps({"streaming": run_streaming(args, args.all_hbm), "workload": workload_label(args)}))
    elif args.exchange:
        args.all_hbm = True
        run_exchange(args)
    elif args.via_peer and args.two_processes:
        run_peer_two_processes(args)
    elif args.via_peer:
        run_peer(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
