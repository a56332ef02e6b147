"""ctypes binding of libflowpool.so: the same calls as include/flowpool.h, argument marshalling only.

Device buffers are passed as integer addresses (torch tensors' data_ptr()); host arrays as numpy.
There is no fallback: if the shared library is missing or cannot be loaded, importing this module fails.
"""
import ctypes as C
import os

import numpy as np

from .build import SO, build

FT_BF16, FT_F32 = 0, 1
FT_RING_SORTED, FT_RING_SHUFFLED = 0, 1
FT_BIND_IDENTITY, FT_BIND_PERMUTED = 0, 1
FT_PLAN_ALLOW_UNWRITTEN, FT_PLAN_SORT_DECREASING, FT_PLAN_COST_SUMSQ, FT_PLAN_ZIGZAG_CARRY, FT_PLAN_AUTO_K = 1, 2, 4, 8, 16
FT_NOALLOC_MAX_SPANS = 4096

STATUS = {
    0: "OK", -1: "INVALID_ARG", -2: "POOL_EXHAUSTED", -3: "UNKNOWN_SAMPLE", -4: "ALREADY_WRITTEN",
    -5: "NOT_READY", -6: "TOO_LONG", -7: "BAD_GVA", -8: "PLACEHOLDER_MISMATCH", -9: "BAD_TOKEN_ID",
    -10: "SLOT_IN_USE", -11: "CAPACITY", -12: "CUDA", -13: "TIMEOUT",
}

EXPORTS = (
    "pool_create", "pool_register_samples", "pool_write_embeddings", "pool_write_embeddings_noalloc",
    "pool_plan_microbatches", "plan_summary",
    "plan_arrays", "plan_destroy", "pool_gather_packed", "pool_gather_list", "pool_set_span_grids", "pool_gather_padded", "pool_embed_grad", "pool_free", "pool_status", "pool_stats",
    "pool_ready_count", "pool_take_ready", "pool_backing", "pool_ipc_export", "pool_ipc_open", "pool_ipc_close", "pool_export_mapping", "pool_import_mapping", "pool_export_samples", "pool_import_samples",
    "pool_get_tuning", "pool_set_tuning", "pool_profile_enable", "pool_profile_read", "pool_debug_span_pages", "pool_debug_ring", "pool_debug_translate", "pool_destroy", "flowpool_last_cuda_error",
)


class FlowpoolError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        detail = ""
        if code == -12:
            detail = ": " + (lib().flowpool_last_cuda_error() or b"").decode()
        super().__init__(f"{where}: FT_ERR_{STATUS.get(code, code)}{detail}")


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


class PoolStats(C.Structure):
    _fields_ = [(k, C.c_uint64) for k in (
        "pages_total", "pages_free", "hbm_pages", "host_pages", "text_pages_total", "text_pages_free",
        "live_samples", "live_spans", "bytes_written", "bytes_gathered", "gpu_launches")]


TUNING_FIELDS = ("dev_ctas_per_sm", "scatter_ctas_per_sm", "scatter_group", "chunk_shift", "host_ctas", "host_store_ctas",
                 "gather_unroll", "grad_ctas_per_sm", "grad_hot_threshold", "remote_ctas", "peers_remote", "scatter_smem_carveout", "gather_smem_carveout",
                 "bulk_wait_limit_us", "bulk_timeout_test", "host_copy_engine")


class Tuning(C.Structure):
    _fields_ = [(k, C.c_uint32) for k in TUNING_FIELDS]


class KernelTime(C.Structure):
    _fields_ = [("ms", C.c_double), ("launches", C.c_uint64)]


KERNEL_CLASSES = ("gather_device", "gather_host", "scatter_device", "scatter_host", "embed_grad", "gather_remote")

IPC_HANDLES_BYTES = 2 * 64 + 8   # ft_ipc_handles


def ipc_open(handles: bytes):
    """Maps a peer process's slabs into this process: (rc, hbm_base, text_base)."""
    buf = (C.c_uint8 * IPC_HANDLES_BYTES).from_buffer_copy(handles)
    a, b = C.c_void_p(), C.c_void_p()
    rc = lib().pool_ipc_open(buf, C.byref(a), C.byref(b))
    return rc, a.value or 0, b.value or 0


def ipc_close(hbm_base: int, text_base: int):
    return lib().pool_ipc_close(hbm_base or None, text_base or None)


_lib = None


def lib():
    """The loaded shared library (built in-tree on first use when nvcc is available)."""
    global _lib
    if _lib is None:
        if not os.path.exists(SO):
            build()
        _lib = C.CDLL(SO)
        P, u32, u64, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int32
        sig = {
            "pool_create": [P, P, P, P],
            "pool_register_samples": [P, u32, P, P, P, P, P, P, P],
            "pool_write_embeddings": [P, u32, P, P, P, P, u32, P],
            "pool_write_embeddings_noalloc": [P, u32, P, P, P, P, u32, P],
            "pool_plan_microbatches": [P, P, u32, P, P, P],
            "plan_summary": [P, P, P, P],
            "plan_arrays": [P] * 13,
            "plan_destroy": [P],
            "pool_gather_packed": [P, P, u32, u32, P, u32, P, P, P, P],
            "pool_gather_list": [P, P, P, u32, P, u32, P, P, P, P],
            "pool_set_span_grids": [P, u32, P, P, P, P],
            "pool_gather_padded": [P, P, u32, u32, P, u32, i32, P, P, P, P, P, P, P],
            "pool_embed_grad": [P, P, u32, u32, u32, P, P, u32, P],
            "pool_free": [P, P, u32, P],
            "pool_status": [P, P, P],
            "pool_stats": [P, P],
            "pool_ready_count": [P, P, P],
            "pool_take_ready": [P, u64, u32, P, P, P],
            "pool_backing": [P, P, P, P],
            "pool_export_mapping": [P, P, u64, P],
            "pool_import_mapping": [P, P, u64, P, P, P],
            "pool_export_samples": [P, P, u32, P, u64, P, P],
            "pool_import_samples": [P, P, u32, P, u64, P],
            "pool_ipc_export": [P, P],
            "pool_ipc_open": [P, P, P],
            "pool_ipc_close": [P, P],
            "pool_get_tuning": [P, P],
            "pool_set_tuning": [P, P],
            "pool_profile_enable": [P, i32],
            "pool_profile_read": [P, P],
            "pool_debug_span_pages": [P, u32, u32, P, u32, P],
            "pool_debug_ring": [P, P, u64, P],
            "pool_debug_translate": [P, P, u32, P, P, P, P],
            "pool_destroy": [P],
        }
        for name, argtypes in sig.items():
            fn = getattr(_lib, name)
            fn.argtypes, fn.restype = argtypes, i32
        _lib.flowpool_last_cuda_error.restype = C.c_char_p
        _lib.flowpool_last_cuda_error.argtypes = []
    return _lib


def _u32(a):
    return np.ascontiguousarray(a, dtype=np.uint32)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class Plan:
    def __init__(self, handle, n, n_ranks):
        self.h, self.n, self.n_ranks = handle, n, n_ranks

    def summary(self):
        n_mb, tot, mx = C.c_uint32(), C.c_uint64(), C.c_uint32()
        rc = lib().plan_summary(self.h, C.byref(n_mb), C.byref(tot), C.byref(mx))
        if rc:
            raise FlowpoolError(rc, "plan_summary")
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
        rc = lib().plan_arrays(self.h, *[_p(v) for v in a.values()])
        if rc:
            raise FlowpoolError(rc, "plan_arrays")
        a["n_mb"] = n_mb
        return a

    def destroy(self):
        if self.h:
            lib().plan_destroy(self.h)
            self.h = None


class Pool:
    """Thin handle around ft_pool.  Every method returns the library's int32 status unchanged
    (0 = OK); nothing is computed on the Python side."""

    def __init__(self, cfg: PoolConfig, hbm_base: int = 0, host_base: int = 0):
        self.cfg = cfg
        self.h = C.c_void_p()
        self.rc = lib().pool_create(C.byref(cfg), hbm_base or None, host_base or None, C.byref(self.h))
        if self.rc != 0:
            self.h = None

    def destroy(self):
        if self.h:
            lib().pool_destroy(self.h)
            self.h = None

    def register_samples(self, slots, seq_len, n_spans, span_pos, span_tokens, input_ids_ptr: int, stream: int = 0):
        slots, seq_len, n_spans = _u32(slots), _u32(seq_len), _u32(n_spans)
        span_pos, span_tokens = _u32(span_pos), _u32(span_tokens)
        return lib().pool_register_samples(self.h, len(slots), _p(slots), _p(seq_len), _p(n_spans), _p(span_pos),
                                           _p(span_tokens), input_ids_ptr or None, stream or None)

    def write_embeddings(self, slots, span_idx, n_tokens, src_ptrs, dtype, stream: int = 0):
        slots, span_idx, n_tokens = _u32(slots), _u32(span_idx), _u32(n_tokens)
        src = np.ascontiguousarray(src_ptrs, dtype=np.uint64)
        return lib().pool_write_embeddings(self.h, len(slots), _p(slots), _p(span_idx), _p(n_tokens), _p(src),
                                           dtype, stream or None)

    def write_embeddings_noalloc(self, slots, span_idx, n_tokens, src_ptrs, dtype, stream: int = 0):
        """pool_write_embeddings_noalloc: same scatter, per-call scratch in the library's fixed device array
        (for callers that may not allocate); at most FT_NOALLOC_MAX_SPANS spans per call."""
        slots, span_idx, n_tokens = _u32(slots), _u32(span_idx), _u32(n_tokens)
        src = np.ascontiguousarray(src_ptrs, dtype=np.uint64)
        return lib().pool_write_embeddings_noalloc(self.h, len(slots), _p(slots), _p(span_idx), _p(n_tokens), _p(src),
                                                   dtype, stream or None)

    def plan_microbatches(self, slots, cfg: PlanConfig, stream: int = 0):
        slots = _u32(slots)
        h = C.c_void_p()
        rc = lib().pool_plan_microbatches(self.h, _p(slots), len(slots), C.byref(cfg), C.byref(h), stream or None)
        return rc, (Plan(h, len(slots), cfg.n_ranks_N) if rc == 0 else None)

    def gather_packed(self, plan: Plan, mb_begin, mb_end, table_ptr: int, vocab: int, out_ptr: int, cu_ptr: int,
                      pos_ptr: int, stream: int = 0):
        return lib().pool_gather_packed(self.h, plan.h, mb_begin, mb_end, table_ptr or None, vocab, out_ptr or None,
                                        cu_ptr or None, pos_ptr or None, stream or None)

    def gather_list(self, plan: Plan, mb_list, table_ptr: int, vocab: int, out_ptr: int, cu_ptr: int, pos_ptr: int,
                    stream: int = 0):
        mb_list = _u32(mb_list)
        return lib().pool_gather_list(self.h, plan.h, _p(mb_list), len(mb_list), table_ptr or None, vocab, out_ptr or None,
                                      cu_ptr or None, pos_ptr or None, stream or None)

    def set_span_grids(self, slots, span_idx, grids, stream: int = 0):
        slots, span_idx = _u32(slots), _u32(span_idx)
        grids = np.ascontiguousarray(np.asarray(grids, dtype=np.uint32).reshape(-1, 3))
        return lib().pool_set_span_grids(self.h, len(slots), _p(slots), _p(span_idx), _p(grids), stream or None)

    def gather_padded(self, plan: Plan, mb_begin, mb_end, table_ptr: int, vocab: int, pad_id: int, out_ptr: int,
                      cu_ptr: int, pos3_ptr: int, ids_ptr: int, labels_ptr: int, mask_ptr: int, stream: int = 0):
        return lib().pool_gather_padded(self.h, plan.h, mb_begin, mb_end, table_ptr or None, vocab, pad_id, out_ptr or None,
                                        cu_ptr or None, pos3_ptr or None, ids_ptr or None, labels_ptr or None,
                                        mask_ptr or None, stream or None)

    def embed_grad(self, plan: Plan, mb_begin, mb_end, padded, grad_out_ptr: int, grad_table_ptr: int, vocab: int,
                   stream: int = 0):
        return lib().pool_embed_grad(self.h, plan.h, mb_begin, mb_end, 1 if padded else 0, grad_out_ptr or None,
                                     grad_table_ptr or None, vocab, stream or None)

    def free(self, slots, stream: int = 0):
        slots = _u32(slots)
        return lib().pool_free(self.h, _p(slots), len(slots), stream or None)

    def status(self):
        code, detail = C.c_int32(), C.c_uint64()
        rc = lib().pool_status(self.h, C.byref(code), C.byref(detail))
        if rc:
            raise FlowpoolError(rc, "pool_status")
        return code.value, detail.value

    def stats(self):
        s = PoolStats()
        rc = lib().pool_stats(self.h, C.byref(s))
        if rc:
            raise FlowpoolError(rc, "pool_stats")
        return {k: getattr(s, k) for k, _ in PoolStats._fields_}

    def ready_count(self):
        n, t = C.c_uint32(), C.c_uint64()
        rc = lib().pool_ready_count(self.h, C.byref(n), C.byref(t))
        if rc:
            raise FlowpoolError(rc, "pool_ready_count")
        return n.value, t.value

    def take_ready(self, min_tokens, max_samples):
        out = np.zeros(max(1, max_samples), np.uint32)
        n, t = C.c_uint32(), C.c_uint64()
        rc = lib().pool_take_ready(self.h, min_tokens, max_samples, _p(out), C.byref(n), C.byref(t))
        return rc, out[: n.value].copy(), t.value

    def backing(self):
        """(hbm_base, host_base as the device sees it, text_base) of this pool's slabs."""
        a, b, c = C.c_void_p(), C.c_void_p(), C.c_void_p()
        rc = lib().pool_backing(self.h, C.byref(a), C.byref(b), C.byref(c))
        if rc:
            raise FlowpoolError(rc, "pool_backing")
        return a.value or 0, b.value or 0, c.value or 0

    def ipc_export(self):
        """Shareable handles (bytes) of this pool's HBM slab and text frames, for a consumer in another process."""
        buf = (C.c_uint8 * IPC_HANDLES_BYTES)()
        rc = lib().pool_ipc_export(self.h, buf)
        return rc, bytes(buf)

    def export_mapping(self):
        n = C.c_uint64()
        rc = lib().pool_export_mapping(self.h, None, 0, C.byref(n))
        if rc:
            return rc, None
        buf = np.zeros(n.value, np.uint8)
        rc = lib().pool_export_mapping(self.h, _p(buf), n.value, C.byref(n))
        return rc, buf

    def import_mapping(self, blob, peer_hbm_base, peer_host_base, peer_text_base):
        blob = np.ascontiguousarray(blob, dtype=np.uint8)
        return lib().pool_import_mapping(self.h, _p(blob), len(blob), peer_hbm_base or None, peer_host_base or None,
                                         peer_text_base or None)

    def export_samples(self, slots, stream: int = 0):
        slots = _u32(slots)
        n = C.c_uint64()
        rc = lib().pool_export_samples(self.h, _p(slots), len(slots), None, 0, C.byref(n), stream or None)
        if rc:
            return rc, None
        buf = np.zeros(n.value, np.uint8)
        rc = lib().pool_export_samples(self.h, _p(slots), len(slots), _p(buf), n.value, C.byref(n), stream or None)
        return rc, buf

    def import_samples(self, local_slots, blob, stream: int = 0):
        local_slots = _u32(local_slots)
        blob = np.ascontiguousarray(blob, dtype=np.uint8)
        return lib().pool_import_samples(self.h, _p(local_slots), len(local_slots), _p(blob), len(blob), stream or None)

    def get_tuning(self):
        t = Tuning()
        rc = lib().pool_get_tuning(self.h, C.byref(t))
        if rc:
            raise FlowpoolError(rc, "pool_get_tuning")
        return {k: getattr(t, k) for k in TUNING_FIELDS}

    def set_tuning(self, **fields):
        """pool_set_tuning: the named knobs, every other one at its default."""
        t = Tuning()
        for k, v in fields.items():
            if k not in TUNING_FIELDS:
                raise KeyError(k)
            setattr(t, k, int(v))
        return lib().pool_set_tuning(self.h, C.byref(t))

    def profile_enable(self, on=True):
        return lib().pool_profile_enable(self.h, 1 if on else 0)

    def profile_read(self):
        out = (KernelTime * len(KERNEL_CLASSES))()
        rc = lib().pool_profile_read(self.h, out)
        if rc:
            raise FlowpoolError(rc, "pool_profile_read")
        return {k: {"ms": out[i].ms, "launches": out[i].launches} for i, k in enumerate(KERNEL_CLASSES)}

    def span_pages(self, slot, span, cap=1 << 16):
        out = np.zeros(cap, np.uint64)
        n = C.c_uint32()
        rc = lib().pool_debug_span_pages(self.h, slot, span, _p(out), cap, C.byref(n))
        return rc, out[: n.value].copy()

    def ring(self):
        total = self.cfg.hbm_pages + self.cfg.host_pages
        out = np.zeros(total, np.uint32)
        n = C.c_uint64()
        rc = lib().pool_debug_ring(self.h, _p(out), total, C.byref(n))
        if rc:
            raise FlowpoolError(rc, "pool_debug_ring")
        return out[: n.value].copy()

    def translate(self, gvas):
        g = np.ascontiguousarray(gvas, dtype=np.uint64)
        kind, frame = np.zeros(len(g), np.uint32), np.zeros(len(g), np.uint64)
        off, st = np.zeros(len(g), np.uint64), np.zeros(len(g), np.int32)
        rc = lib().pool_debug_translate(self.h, _p(g), len(g), _p(kind), _p(frame), _p(off), _p(st))
        if rc:
            raise FlowpoolError(rc, "pool_debug_translate")
        return st, kind, frame, off
