"""ctypes front end of the C oracle (flowpool_oracle.c) -- TEST INFRASTRUCTURE.

Builds the oracle with gcc on first use and wraps its calls with numpy
arrays.  No arithmetic of the method lives in this file; it only marshals.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "flowpool_oracle.c")
_SO = os.path.join(_HERE, "libflowpool_oracle.so")

STATUS = {
    0: "OK", -1: "INVALID_ARG", -2: "POOL_EXHAUSTED", -3: "UNKNOWN_SAMPLE", -4: "ALREADY_WRITTEN",
    -5: "NOT_READY", -6: "TOO_LONG", -7: "BAD_GVA", -8: "PLACEHOLDER_MISMATCH", -9: "BAD_TOKEN_ID",
    -10: "SLOT_IN_USE", -11: "CAPACITY", -12: "CUDA", -13: "TIMEOUT",
}


class PoolConfig(C.Structure):
    _fields_ = [
        ("page_bytes", C.c_uint64), ("hbm_pages", C.c_uint64), ("host_pages", C.c_uint64),
        ("max_text_tokens", C.c_uint64), ("ring_seed", C.c_uint64), ("bind_seed", C.c_uint64),
        ("gva_hbm_start", C.c_uint64), ("gva_host_start", C.c_uint64), ("max_size", C.c_uint64),
        ("hidden", C.c_uint32), ("max_samples", C.c_uint32), ("max_spans_per_sample", C.c_uint32),
        ("max_pages_per_span", C.c_uint32), ("max_seq_len", C.c_uint32),
        ("placeholder_id", C.c_int32), ("ring_order", C.c_uint32), ("bind_order", C.c_uint32),
        ("world_size", C.c_uint32), ("rank", C.c_uint32), ("max_imported_pages", C.c_uint64),
    ]


class PlanConfig(C.Structure):
    _fields_ = [
        ("coef_A", C.c_uint64), ("coef_B", C.c_uint64), ("budget_L", C.c_uint32),
        ("n_buckets_K", C.c_uint32), ("n_ranks_N", C.c_uint32), ("flags", C.c_uint32),
    ]


def build_oracle(force=False):
    """Compile the C oracle into a shared object next to its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-shared", "-fPIC", "-o", _SO, _SRC])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_oracle())
        _lib.oracle_page_gva.restype = C.c_uint64
        _lib.oracle_page_gva.argtypes = [C.c_void_p, C.c_uint64]
        _lib.oracle_segment_base.restype = C.c_uint64
        _lib.oracle_segment_base.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32]
        _lib.oracle_f32_to_bf16_rne.restype = C.c_uint16
        _lib.oracle_f32_to_bf16_rne.argtypes = [C.c_uint32]
        _lib.oracle_cost_int.restype = C.c_uint64
        _lib.oracle_cost_int.argtypes = [C.c_uint64] * 4
        _lib.oracle_pool_backing.restype = C.c_void_p
        _lib.oracle_pool_backing.argtypes = [C.c_void_p, C.c_uint32]
        _lib.oracle_bestfit_segment_tree.restype = C.c_uint32
        _lib.oracle_balance.restype = None
    return _lib


def _u32(a):
    return np.ascontiguousarray(a, dtype=np.uint32)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def f32_to_bf16_rne(bits):
    return int(lib().oracle_f32_to_bf16_rne(int(bits) & 0xFFFFFFFF))


def cost_int(A, B, sum_len, lmax):
    return int(lib().oracle_cost_int(A, B, sum_len, lmax))


def bestfit_segment_tree(lengths, L, l_min):
    lengths = _u32(lengths)
    out = np.zeros(len(lengths), dtype=np.uint32)
    n_mb = lib().oracle_bestfit_segment_tree(C.c_uint32(len(lengths)), _p(lengths), C.c_uint32(L),
                                             C.c_uint32(l_min), _p(out))
    return int(n_mb), out


def balance(costs, K, N, carry=0):
    """Algorithm 1 lines 12-27 on explicit costs -> dict(bucket, rank, rank_mb_off, rank_mbs).
    carry=1: the zig-zag position and direction carry over from bucket to bucket (variant)."""
    costs = np.ascontiguousarray(costs, dtype=np.uint64)
    m = len(costs)
    out = {"bucket": np.zeros(m, np.uint32), "rank": np.zeros(m, np.uint32),
           "rank_mb_off": np.zeros(N + 1, np.uint32), "rank_mbs": np.zeros(m, np.uint32)}
    lib().oracle_balance(C.c_uint32(m), _p(costs), C.c_uint32(K), C.c_uint32(N), C.c_int(carry), *[_p(v) for v in out.values()])
    return out


class OraclePlan:
    def __init__(self, handle, n, n_ranks):
        self.h = handle
        self.n = n
        self.n_ranks = n_ranks

    def summary(self):
        n_mb, tot, mx = C.c_uint32(), C.c_uint64(), C.c_uint32()
        rc = lib().oracle_plan_summary(self.h, C.byref(n_mb), C.byref(tot), C.byref(mx))
        assert rc == 0
        return n_mb.value, tot.value, mx.value

    def arrays(self):
        n_mb = self.summary()[0]
        n, N = self.n, self.n_ranks
        a = {
            "mb_sample_off": np.zeros(n_mb + 1, np.uint32), "mb_samples": np.zeros(n, np.uint32),
            "mb_tokens": np.zeros(n_mb, np.uint32), "mb_lmax": np.zeros(n_mb, np.uint32),
            "mb_residual": np.zeros(n_mb, np.uint32), "mb_cost": np.zeros(n_mb, np.uint64),
            "mb_bucket": np.zeros(n_mb, np.uint32), "mb_rank": np.zeros(n_mb, np.uint32),
            "rank_mb_off": np.zeros(N + 1, np.uint32), "rank_mbs": np.zeros(n_mb, np.uint32),
            "sample_cost": np.zeros(n, np.uint64), "sample_mb": np.zeros(n, np.uint32),
        }
        rc = lib().oracle_plan_arrays(self.h, *[_p(v) for v in a.values()])
        assert rc == 0
        a["n_mb"] = n_mb
        return a

    def destroy(self):
        if self.h:
            lib().oracle_plan_destroy(self.h)
            self.h = None


def plan_from_lengths(lengths, cfg, slots=None):
    """Algorithm 1 on bare lengths (no pool).  Returns (status, OraclePlan|None)."""
    lengths = _u32(lengths)
    slots_a = None if slots is None else _u32(slots)
    h = C.c_void_p()
    rc = lib().oracle_plan_from_lengths(_p(slots_a), _p(lengths), C.c_uint32(len(lengths)), C.byref(cfg), C.byref(h))
    return rc, (OraclePlan(h, len(lengths), cfg.n_ranks_N) if rc == 0 else None)


class OraclePool:
    """Host-memory pool with the same call sequence as the CUDA library."""

    def __init__(self, cfg):
        self.cfg = cfg
        self.h = C.c_void_p()
        self.rc = lib().oracle_pool_create(C.byref(cfg), C.byref(self.h))
        if self.rc != 0:
            self.h = None

    def destroy(self):
        if self.h:
            lib().oracle_pool_destroy(self.h)
            self.h = None

    def register_samples(self, slots, seq_len, n_spans, span_pos, span_tokens, input_ids):
        slots, seq_len, n_spans = _u32(slots), _u32(seq_len), _u32(n_spans)
        span_pos, span_tokens = _u32(span_pos), _u32(span_tokens)
        ids = np.ascontiguousarray(input_ids, dtype=np.int32)
        return lib().oracle_pool_register_samples(self.h, C.c_uint32(len(slots)), _p(slots), _p(seq_len), _p(n_spans),
                                                  _p(span_pos), _p(span_tokens), _p(ids))

    def write_embeddings(self, slots, span_idx, n_tokens, srcs, dtype):
        """srcs: list of contiguous numpy arrays (uint16 bf16 bits, or float32/uint32)."""
        slots, span_idx, n_tokens = _u32(slots), _u32(span_idx), _u32(n_tokens)
        srcs = [np.ascontiguousarray(s) for s in srcs]
        ptrs = (C.c_void_p * max(1, len(srcs)))(*[s.ctypes.data for s in srcs])
        return lib().oracle_pool_write_embeddings(self.h, C.c_uint32(len(slots)), _p(slots), _p(span_idx),
                                                  _p(n_tokens), ptrs, C.c_uint32(dtype))

    def plan_microbatches(self, slots, cfg):
        slots = _u32(slots)
        h = C.c_void_p()
        rc = lib().oracle_pool_plan_microbatches(self.h, _p(slots), C.c_uint32(len(slots)), C.byref(cfg), C.byref(h))
        return rc, (OraclePlan(h, len(slots), cfg.n_ranks_N) if rc == 0 else None)

    def gather_packed(self, plan, mb_begin, mb_end, table, out, cu, pos):
        """table: uint16 [vocab, H]; out: uint16 [rows, H]; cu, pos: int32 arrays (written in place)."""
        return lib().oracle_pool_gather_packed(self.h, plan.h, C.c_uint32(mb_begin), C.c_uint32(mb_end), _p(table),
                                               C.c_uint32(table.shape[0]), _p(out), _p(cu), _p(pos))

    def gather_list(self, plan, mb_list, table, out, cu, pos):
        """The microbatches of mb_list, in list order (outputs as gather_packed, concatenated)."""
        mb_list = _u32(mb_list)
        return lib().oracle_pool_gather_list(self.h, plan.h, _p(mb_list), C.c_uint32(len(mb_list)), _p(table),
                                             C.c_uint32(table.shape[0]), _p(out), _p(cu), _p(pos))

    def set_span_grids(self, slots, span_idx, grids):
        """grids: [n, 3] (T, H, W) per named span."""
        slots, span_idx = _u32(slots), _u32(span_idx)
        grids = np.ascontiguousarray(np.asarray(grids, dtype=np.uint32).reshape(-1, 3))
        return lib().oracle_pool_set_span_grids(self.h, C.c_uint32(len(slots)), _p(slots), _p(span_idx), _p(grids))

    def gather_padded(self, plan, mb_begin, mb_end, table, pad_id, out, cu, pos3, ids, labels, mask):
        """out: uint16 [n_mb*L, H]; cu: int32; pos3: int32 [3, rows]; ids, labels: int32 [rows]; mask: uint8 [rows]."""
        return lib().oracle_pool_gather_padded(self.h, plan.h, C.c_uint32(mb_begin), C.c_uint32(mb_end), _p(table),
                                               C.c_uint32(table.shape[0]), C.c_int32(pad_id), _p(out), _p(cu), _p(pos3),
                                               _p(ids), _p(labels), _p(mask))

    def embed_grad(self, plan, mb_begin, mb_end, padded, grad_out, grad_table):
        """grad_out: uint16 (bf16 bits) [rows, H]; grad_table: float32 [vocab, H], accumulated in place."""
        return lib().oracle_pool_embed_grad(self.h, plan.h, C.c_uint32(mb_begin), C.c_uint32(mb_end), C.c_int(int(padded)),
                                            _p(grad_out), _p(grad_table), C.c_uint32(grad_table.shape[0]))

    def free(self, slots):
        slots = _u32(slots)
        return lib().oracle_pool_free(self.h, _p(slots), C.c_uint32(len(slots)))

    def status(self):
        code, detail = C.c_int32(), C.c_uint64()
        lib().oracle_pool_status(self.h, C.byref(code), C.byref(detail))
        return code.value, detail.value

    def span_pages(self, slot, span, cap=1 << 16):
        out = np.zeros(cap, np.uint64)
        n = C.c_uint32()
        rc = lib().oracle_pool_debug_span_pages(self.h, C.c_uint32(slot), C.c_uint32(span), _p(out), C.c_uint32(cap), C.byref(n))
        return rc, out[: n.value].copy()

    def free_pages(self):
        a, b = C.c_uint64(), C.c_uint64()
        lib().oracle_pool_free_pages(self.h, C.byref(a), C.byref(b))
        return a.value, b.value

    def ring(self):
        total = self.cfg.hbm_pages + self.cfg.host_pages
        out = np.zeros(total, np.uint32)
        n = C.c_uint64()
        lib().oracle_pool_debug_ring(self.h, _p(out), C.c_uint64(total), C.byref(n))
        return out[: n.value].copy()

    def translate(self, gva):
        kind, frame, off = C.c_uint32(), C.c_uint64(), C.c_uint64()
        rc = lib().oracle_translate(self.h, C.c_uint64(gva), C.byref(kind), C.byref(frame), C.byref(off))
        return rc, kind.value, frame.value, off.value

    def page_gva(self, global_page):
        return int(lib().oracle_page_gva(self.h, C.c_uint64(global_page)))

    def segment_base(self, tier, proc):
        return int(lib().oracle_segment_base(self.h, C.c_uint32(tier), C.c_uint32(proc)))

    def translate_ex(self, gva):
        proc, kind, frame, off = C.c_uint32(), C.c_uint32(), C.c_uint64(), C.c_uint64()
        rc = lib().oracle_translate_ex(self.h, C.c_uint64(gva), C.byref(proc), C.byref(kind), C.byref(frame), C.byref(off))
        return rc, proc.value, kind.value, frame.value, off.value

    def export_mapping(self):
        n = C.c_uint64()
        lib().oracle_pool_export_mapping(self.h, None, C.c_uint64(0), C.byref(n))
        buf = np.zeros(n.value, np.uint8)
        rc = lib().oracle_pool_export_mapping(self.h, _p(buf), C.c_uint64(n.value), C.byref(n))
        return rc, buf

    def import_mapping(self, blob, peer):
        """peer: the OraclePool whose mapping this is (its backing arrays are reached directly: one process)."""
        blob = np.ascontiguousarray(blob, dtype=np.uint8)
        ptrs = [C.c_void_p(lib().oracle_pool_backing(peer.h, C.c_uint32(k))) for k in range(3)] if peer is not None else [None] * 3
        return lib().oracle_pool_import_mapping(self.h, _p(blob), C.c_uint64(len(blob)), *ptrs)

    def export_samples(self, slots):
        slots = _u32(slots)
        n = C.c_uint64()
        rc = lib().oracle_pool_export_samples(self.h, _p(slots), C.c_uint32(len(slots)), None, C.c_uint64(0), C.byref(n))
        if rc:
            return rc, None
        buf = np.zeros(n.value, np.uint8)
        rc = lib().oracle_pool_export_samples(self.h, _p(slots), C.c_uint32(len(slots)), _p(buf), C.c_uint64(n.value), C.byref(n))
        return rc, buf

    def import_samples(self, local_slots, blob):
        local_slots = _u32(local_slots)
        blob = np.ascontiguousarray(blob, dtype=np.uint8)
        return lib().oracle_pool_import_samples(self.h, _p(local_slots), C.c_uint32(len(local_slots)), _p(blob), C.c_uint64(len(blob)))

    def ready_count(self):
        n, t = C.c_uint32(), C.c_uint64()
        lib().oracle_pool_ready_count(self.h, C.byref(n), C.byref(t))
        return n.value, t.value

    def take_ready(self, min_tokens, max_samples):
        out = np.zeros(max(1, max_samples), np.uint32)
        n, t = C.c_uint32(), C.c_uint64()
        rc = lib().oracle_pool_take_ready(self.h, C.c_uint64(min_tokens), C.c_uint32(max_samples), _p(out), C.byref(n), C.byref(t))
        return rc, out[: n.value].copy(), t.value

    def backing(self, kind):
        """numpy view (uint8) of a tier's backing frames: 0 HBM, 1 DRAM."""
        pages = self.cfg.hbm_pages if kind == 0 else self.cfg.host_pages
        nbytes = pages * self.cfg.page_bytes
        addr = lib().oracle_pool_backing(self.h, C.c_uint32(kind))
        return np.ctypeslib.as_array((C.c_uint8 * nbytes).from_address(addr))
