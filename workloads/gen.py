"""Seeded, counter-based synthetic workloads (inputs only).

Every random quantity is a pure function of (seed, stream, index) through one
stateless 64-bit integer mixer, so any piece can be regenerated anywhere --
host or device, whole or sampled -- with identical bits.

* Lengths, span counts and span positions are drawn once on the host (numpy,
  float64 for the log-normal draws) and handed to both implementations as
  the same integer arrays.
* Embedding values are "bf16 N(0,1)" realised as an Irwin-Hall(4) sum: the
  four 16-bit fields of the hash, minus 131070, converted exactly to fp32 and
  multiplied once by the fp32 reciprocal standard deviation, then rounded to
  bf16 by the tensor library (no NaNs occur, so every rounding mode question
  is moot: one exact int->float conversion, one IEEE multiply, one RNE).
  Generated with torch ops, so the same code runs on CPU and on a CUDA device.
"""
from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np
import torch

_M64 = (1 << 64) - 1
_G = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

# stream ids
S_NTOK, S_TEXT, S_NSPAN, S_POS, S_IDS, S_EMB, S_TABLE, S_PERM, S_FRAMES, S_FREE, S_GRID, S_GRAD = range(1, 13)

# fp32 reciprocal of the standard deviation of a sum of four uniform 16-bit integers
_IH_SCALE_BITS = 0x37DDB3D7

CONFIG_NAMES = ("tiny", "image_mix_7b", "video_heavy", "host_tier_stress", "frag_sweep")


def _pymix(z: int) -> int:
    z = (z + _G) & _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, stream: int, a: int = 0, b: int = 0) -> int:
    return _pymix(_pymix(_pymix(_pymix(seed) ^ stream) ^ a) ^ b)


def _mix_np(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64)
    with np.errstate(over="ignore"):
        z = z + np.uint64(_G)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_C1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_C2)
        return z ^ (z >> np.uint64(31))


def _signed(c: int) -> int:
    return c - (1 << 64) if c >= (1 << 63) else c


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix_torch(z: torch.Tensor) -> torch.Tensor:
    """Same mixer on an int64 tensor (two's-complement wrap-around multiply)."""
    z = z + _signed(_G)
    z = (z ^ _lsr(z, 30)) * _signed(_C1)
    z = (z ^ _lsr(z, 27)) * _signed(_C2)
    return z ^ _lsr(z, 31)


def hash_np(key: int, idx) -> np.ndarray:
    idx = np.asarray(idx, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix_np(idx + np.uint64(key))


def u01(key: int, idx) -> np.ndarray:
    return (hash_np(key, idx) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def randint(key: int, idx, lo: int, hi: int) -> np.ndarray:
    """Uniform integers in [lo, hi], inclusive."""
    return (lo + np.floor(u01(key, idx) * (hi - lo + 1))).astype(np.int64)


def lognormal(key: int, idx, median: float, sigma: float) -> np.ndarray:
    idx = np.asarray(idx, dtype=np.uint64)
    u1 = 1.0 - u01(key, idx * np.uint64(2))
    u2 = u01(key, idx * np.uint64(2) + np.uint64(1))
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return median * np.exp(sigma * z)


def permutation(key: int, n: int) -> np.ndarray:
    """A seeded permutation (argsort of hashes); inputs only, unrelated to the pool's own shuffles."""
    return np.argsort(hash_np(key, np.arange(n)), kind="stable")


@dataclass
class Workload:
    name: str
    seed: int
    hidden: int
    page_bytes: int
    vocab: int
    placeholder_id: int
    src_dtype: int                     # 0 = bf16 source, 1 = fp32 source (cast on write)
    seq_len: np.ndarray                # [n] uint32
    n_spans: np.ndarray                # [n] uint32
    span_off: np.ndarray               # [n+1] int64, into span_pos/span_tokens
    span_pos: np.ndarray               # [S] uint32, sequence coordinates
    span_tokens: np.ndarray            # [S] uint32
    hbm_pages: int
    host_pages: int
    ring_order: int                    # 0 sorted, 1 shuffled
    bind_order: int                    # 0 identity, 1 permuted
    budget_L: int
    coef_A: int
    coef_B: int
    n_buckets_K: int = 4
    n_ranks_N: int = 8
    write_calls: List[List[Tuple[int, int]]] = field(default_factory=list)  # per call: (sample, span_idx)
    plan_order: List[int] = field(default_factory=list)                     # sample ids, completion order
    max_spans_per_sample: int = 1
    max_pages_per_span: int = 1
    max_seq_len: int = 1
    id_skew: str = "uniform"          # text-token ids: "uniform", or "zipf" (P(id = k) roughly proportional to 1 / (k + 1))

    @property
    def n_samples(self) -> int:
        return len(self.seq_len)

    @property
    def row_bytes(self) -> int:
        return 2 * self.hidden

    def spans_of(self, s: int):
        a, b = int(self.span_off[s]), int(self.span_off[s + 1])
        return self.span_pos[a:b], self.span_tokens[a:b]

    def pages_of_span(self, n_tokens: int) -> int:
        return -(-int(n_tokens) * self.row_bytes // self.page_bytes)

    @property
    def total_tokens(self) -> int:
        return int(self.seq_len.astype(np.int64).sum())

    @property
    def total_vision_tokens(self) -> int:
        return int(self.span_tokens.astype(np.int64).sum())

    @property
    def total_text_tokens_capacity(self) -> int:
        """Text-page budget in tokens: every sample rounded up to whole 1024-id pages."""
        return int(((self.seq_len.astype(np.int64) + 1023) // 1024).sum()) * 1024


def _assemble(name, seed, hidden, page_bytes, text_len, tokens_per_span, **kw) -> Workload:
    """text_len[n]; tokens_per_span: list of per-sample arrays.  Span positions: sorted uniform draws in
    [0, T] (text coordinates, repeats allowed => adjacent runs), shifted by the vision tokens before them."""
    n = len(text_len)
    n_spans = np.array([len(t) for t in tokens_per_span], dtype=np.uint32)
    span_off = np.zeros(n + 1, dtype=np.int64)
    span_off[1:] = np.cumsum(n_spans)
    span_pos = np.zeros(int(span_off[-1]), dtype=np.uint32)
    span_tokens = np.zeros(int(span_off[-1]), dtype=np.uint32)
    seq_len = np.zeros(n, dtype=np.uint32)
    kpos = stream_key(seed, S_POS)
    for s in range(n):
        toks = np.asarray(tokens_per_span[s], dtype=np.int64)
        a = int(span_off[s])
        draws = np.sort(randint(kpos, a + np.arange(len(toks)), 0, int(text_len[s])))
        before = np.concatenate([[0], np.cumsum(toks)[:-1]]) if len(toks) else np.zeros(0, np.int64)
        span_pos[a:a + len(toks)] = draws + before
        span_tokens[a:a + len(toks)] = toks
        seq_len[s] = int(text_len[s]) + int(toks.sum())
    vocab = 32768
    w = Workload(name=name, seed=seed, hidden=hidden, page_bytes=page_bytes, vocab=vocab, placeholder_id=vocab - 1,
                 src_dtype=kw.pop("src_dtype", 0), seq_len=seq_len, n_spans=n_spans, span_off=span_off,
                 span_pos=span_pos, span_tokens=span_tokens, hbm_pages=0, host_pages=0,
                 ring_order=kw.pop("ring_order", 0), bind_order=kw.pop("bind_order", 1), budget_L=kw.pop("budget_L"),
                 coef_A=0, coef_B=1)
    w.coef_A = kw.pop("coef_A", w.budget_L)
    w.max_spans_per_sample = max(1, int(n_spans.max()) if n else 1)
    w.max_pages_per_span = max(1, max((w.pages_of_span(t) for t in span_tokens), default=1))
    w.max_seq_len = max(1, int(seq_len.max()) if n else 1)
    assert not kw, kw
    return w


def _pages_needed(w: Workload) -> int:
    return int(sum(w.pages_of_span(t) for t in w.span_tokens))


def _calls_by_sample(order, per_call, w):
    calls = []
    for i in range(0, len(order), per_call):
        calls.append([(int(s), j) for s in order[i:i + per_call] for j in range(int(w.n_spans[s]))])
    return calls


def make_workload(name: str, n_samples: int = None, page_bytes: int = None, hidden: int = None,
                  all_hbm: bool = False, pool_bytes: int = None, id_skew: str = "uniform") -> Workload:
    """The five configurations; n_samples / hidden / page_bytes shrink them for parity tests."""
    if name == "tiny":  # seed 0
        seed, n = 0, n_samples or 16
        H, PS = hidden or 1024, page_bytes or 64 << 10
        idx = np.arange(n)
        ntok = randint(stream_key(seed, S_NTOK), idx, 64, 256)
        text = randint(stream_key(seed, S_TEXT), idx, 32, 512)
        w = _assemble(name, seed, H, PS, text, [[t] for t in ntok], budget_L=4096)
        w.hbm_pages, w.host_pages = max(128, _pages_needed(w) + 8), 0
        w.write_calls = _calls_by_sample(list(range(n)), n, w)
        w.plan_order = list(range(n))
    elif name == "image_mix_7b":  # seed 1
        seed, n = 1, n_samples or 512
        H, PS = hidden or 3584, page_bytes or 2 << 20
        idx = np.arange(n)
        nsp = randint(stream_key(seed, S_NSPAN), idx, 1, 4)
        text = randint(stream_key(seed, S_TEXT), idx, 128, 4096)
        kt = stream_key(seed, S_NTOK)
        toks, c = [], 0
        for s in range(n):
            v = np.clip(np.rint(lognormal(kt, c + np.arange(nsp[s]), 1024.0, 0.7)), 256, 4096).astype(np.int64)
            toks.append(v)
            c += int(nsp[s])
        w = _assemble(name, seed, H, PS, text, toks, budget_L=32768, coef_A=12 * 3584)
        P = -(-_pages_needed(w) * 102 // 100)
        w.hbm_pages = P * 8 // 10
        w.host_pages = P - w.hbm_pages
        w.write_calls = _calls_by_sample(list(range(n)), 32, w)
        w.plan_order = list(range(n))
    elif name == "video_heavy":  # seed 2
        seed, n = 2, n_samples or 128
        H, PS = hidden or 4096, page_bytes or 2 << 20
        idx = np.arange(n)
        frames = randint(stream_key(seed, S_FRAMES), idx, 8, 64)
        text = randint(stream_key(seed, S_TEXT), idx, 256, 2048)
        w = _assemble(name, seed, H, PS, text, [[256] * int(f) for f in frames], budget_L=131072)
        w.hbm_pages, w.host_pages = _pages_needed(w) + 16, 0
        order = [int(x) for x in permutation(stream_key(seed, S_PERM), n)]  # producer completion order
        w.write_calls = _calls_by_sample(order, 8, w)
        w.plan_order = order
    elif name == "host_tier_stress":  # seed 3
        seed, n = 3, n_samples or 256
        H, PS = hidden or 8192, page_bytes or 2 << 20
        idx = np.arange(n)
        ntok = randint(stream_key(seed, S_NTOK), idx, 2048, 8192)
        text = randint(stream_key(seed, S_TEXT), idx, 128, 2048)
        w = _assemble(name, seed, H, PS, text, [[t] for t in ntok], budget_L=65536, src_dtype=1, ring_order=1)
        P = _pages_needed(w) + 8
        P += P & 1
        w.hbm_pages = w.host_pages = P // 2
        w.write_calls = _calls_by_sample(list(range(n)), 16, w)
        w.plan_order = list(range(n))
    elif name == "frag_sweep":  # seed 4: the sample stream; the churn schedule comes from admit_free_schedule
        seed, n = 4, n_samples or 65536
        H, PS = hidden or 4096, page_bytes or 2 << 20
        idx = np.arange(n)
        ntok = np.clip(np.rint(lognormal(stream_key(seed, S_NTOK), idx, 512.0, 1.0)), 64, 16384).astype(np.int64)
        text = randint(stream_key(seed, S_TEXT), idx, 32, 1024)
        w = _assemble(name, seed, H, PS, text, [[t] for t in ntok], budget_L=32768)
        w.hbm_pages, w.host_pages = (pool_bytes or (64 << 30)) // PS, 0
        w.write_calls, w.plan_order = [], []
    else:
        raise ValueError(name)
    if all_hbm:
        w.hbm_pages, w.host_pages = w.hbm_pages + w.host_pages, 0
    assert id_skew in ("uniform", "zipf")
    w.id_skew = id_skew
    return w


def admit_free_schedule(w: Workload, cycles: int = 10):
    """Churn script for the fragmentation sweep: `cycles` x { admit the next samples of the stream, in order,
    while their pages fit; free a seeded-random half of the residents }, then a final admit-until-full.
    Returns (ops, residents): ops = list of ("admit", [samples]) / ("free", [samples]); residents in
    admission order.  Pure bookkeeping on page counts; no pool is touched."""
    free_pages = w.hbm_pages + w.host_pages
    need = [w.pages_of_span(t) for t in w.span_tokens]  # one span per sample in this config
    nxt, residents, ops = 0, [], []
    kfree = stream_key(w.seed, S_FREE)
    for cyc in range(cycles + 1):
        batch = []
        while nxt < w.n_samples and need[nxt] <= free_pages:
            free_pages -= need[nxt]
            batch.append(nxt)
            nxt += 1
        if batch:
            ops.append(("admit", batch))
            residents += batch
        if cyc == cycles:
            break
        h = hash_np(kfree, np.asarray(residents, dtype=np.uint64) + np.uint64(cyc << 32))
        gone = [s for s, x in zip(residents, h) if int(x) & 1]
        if gone:
            ops.append(("free", gone))
            free_pages += sum(need[s] for s in gone)
            gs = set(gone)
            residents = [s for s in residents if s not in gs]
    return ops, residents


# ---------------------------------------------------------------------------------------------
# values
# ---------------------------------------------------------------------------------------------

def input_ids(w: Workload, s: int) -> np.ndarray:
    """int32[seq_len]: ids in [0, vocab-2], uniform or log-uniform (a Zipf-like head: id 0 is the most frequent);
    the placeholder id on every span's run."""
    n = int(w.seq_len[s])
    if w.id_skew == "zipf":
        u = u01(stream_key(w.seed, S_IDS, s), np.arange(n))
        ids = np.clip(np.floor(np.exp(u * np.log(w.vocab - 1.0))).astype(np.int64) - 1, 0, w.vocab - 2).astype(np.int32)
    else:
        ids = randint(stream_key(w.seed, S_IDS, s), np.arange(n), 0, w.vocab - 2).astype(np.int32)
    pos, tok = w.spans_of(s)
    for p, t in zip(pos, tok):
        ids[int(p):int(p) + int(t)] = w.placeholder_id
    return ids


def span_grid(w: Workload, s: int, j: int):
    """Token grid (T, H, W) of span j of sample s, or None (one span in four has none).  W is the largest divisor
    of the tokens of one frame that is at most its square root, T is 2 for every other even-sized span, else 1."""
    n = int(w.spans_of(s)[1][j])
    h = int(hash_np(stream_key(w.seed, S_GRID, s), np.array([j]))[0])
    if h % 4 == 0:
        return None
    T = 2 if (n % 2 == 0 and (h >> 8) % 2 == 0) else 1
    frame = n // T
    W = max(d for d in range(1, int(frame ** 0.5) + 1) if frame % d == 0)
    return T, frame // W, W


def grad_values(w: Workload, row0: int, row1: int, device="cpu") -> torch.Tensor:
    """bf16 [row1-row0, H] stand-in for the gradient w.r.t. the assembled rows row0..row1 of a layout."""
    return _irwin_hall_f32(stream_key(w.seed, S_GRAD), row0 * w.hidden, row1 * w.hidden, device).to(torch.bfloat16).view(row1 - row0, w.hidden)


def _irwin_hall_f32(key: int, e0: int, e1: int, device) -> torch.Tensor:
    idx = torch.arange(e0, e1, dtype=torch.int64, device=device)
    h = _mix_torch(idx + _signed(key))
    s = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + (_lsr(h, 48) & 0xFFFF) - 131070
    scale = torch.tensor([_IH_SCALE_BITS], dtype=torch.int32, device=device).view(torch.float32)
    return s.to(torch.float32) * scale


def special_f32_bits() -> np.ndarray:
    """fp32 bit patterns that stress the cast: signed zeros, infinities, NaNs, denormals, ties, overflow."""
    return np.array([
        0x00000000, 0x80000000, 0x7F800000, 0xFF800000, 0x7FC00000, 0xFFC00001, 0x7F800001, 0xFFFFFFFF,
        0x00000001, 0x00018000, 0x807FFFFF, 0x007FFFFF, 0x3F808000, 0x3F818000, 0x3F808001, 0x3F807FFF,
        0x7F7FFFFF, 0x7F7F7FFF, 0xFF7FFFFF, 0x7F7F8000, 0x00008000, 0x80008000, 0x00008001, 0x7FBFFFFF,
    ], dtype=np.uint32)


def span_values(w: Workload, s: int, j: int, device="cpu", rows=None) -> torch.Tensor:
    """Encoder output of span j of sample s: [n_tokens, H] bf16, or fp32 when w.src_dtype == 1 (then every
    4099-th element of the span is replaced by a special bit pattern).  rows=(r0, r1) restricts to a row range."""
    pos, tok = w.spans_of(s)
    n, H = int(tok[j]), w.hidden
    r0, r1 = (0, n) if rows is None else rows
    key = stream_key(w.seed, S_EMB, s, j)
    x = _irwin_hall_f32(key, r0 * H, r1 * H, device)
    if w.src_dtype == 0:
        return x.to(torch.bfloat16).view(r1 - r0, H)
    e = torch.arange(r0 * H, r1 * H, dtype=torch.int64, device=device)
    tab = torch.from_numpy(special_f32_bits().astype(np.int64)).to(device)
    hit = (e % 4099) == 0
    spec = tab[(e // 4099) % len(tab)]
    bits = torch.where(hit, spec, x.view(torch.int32).to(torch.int64) & 0xFFFFFFFF)
    bits = torch.where(bits >= (1 << 31), bits - (1 << 32), bits).to(torch.int32)
    return bits.view(torch.float32).view(r1 - r0, H)


def embed_table(w: Workload, device="cpu", rows=None) -> torch.Tensor:
    """Text-token embedding table [vocab, H] bf16 (or a row range of it)."""
    r0, r1 = (0, w.vocab) if rows is None else rows
    key = stream_key(w.seed, S_TABLE)
    out = torch.empty((r1 - r0, w.hidden), dtype=torch.bfloat16, device=device)
    step = max(1, (1 << 24) // w.hidden)
    for a in range(r0, r1, step):
        b = min(r1, a + step)
        out[a - r0:b - r0] = _irwin_hall_f32(key, a * w.hidden, b * w.hidden, device).to(torch.bfloat16).view(b - a, w.hidden)
    return out
