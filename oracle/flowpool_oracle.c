/*
 * flowpool_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, single-threaded CPU statement of what the unified-memory-pool
 * hot path computes: GVA layout and page tables (paper Sec. 3.2), the page
 * free ring, the producer write with its optional fp32->bf16 cast, the dynamic
 * packing rule (Algorithm 1, Eq. 3) and the consumer's packed-microbatch
 * assembly.  Arrays and loops only: no scans, no bitmaps, no blocking.  It
 * shares nothing with the CUDA library (no header, no helper, no table); only
 * tests, the smoke check and the benchmark's CPU-baseline leg may use it.
 *
 * Where the paper is silent the fixed rule used here is stated next to the
 * code that applies it ("reading:").  Parts whose result the paper does not
 * determine are marked "parity unpinned": GVA base constants, the page
 * assignment order (free ring), the best-fit tie-break, the bucket rule, the
 * bucket/tie orders of the zig-zag, and the NaN encoding of the cast.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- status codes (same numeric values as the library's public header;
 *      retyped here on purpose, the two sides share no file) ---- */
enum {
  OR_OK = 0,
  OR_ERR_INVALID_ARG = -1,
  OR_ERR_POOL_EXHAUSTED = -2,
  OR_ERR_UNKNOWN_SAMPLE = -3,
  OR_ERR_ALREADY_WRITTEN = -4,
  OR_ERR_NOT_READY = -5,
  OR_ERR_TOO_LONG = -6,
  OR_ERR_BAD_GVA = -7,
  OR_ERR_PLACEHOLDER_MISMATCH = -8,
  OR_ERR_BAD_TOKEN_ID = -9,
  OR_ERR_SLOT_IN_USE = -10,
  OR_ERR_CAPACITY = -11,
  OR_ERR_CUDA = -12,
  OR_ERR_TIMEOUT = -13
};

enum { OR_RING_SORTED = 0, OR_RING_SHUFFLED = 1 };
enum { OR_BIND_IDENTITY = 0, OR_BIND_PERMUTED = 1 };
enum { OR_BF16 = 0, OR_F32 = 1 };
/* plan flags; the last three are variants at points where the paper is silent or could be read otherwise */
enum { OR_PLAN_ALLOW_UNWRITTEN = 1, OR_PLAN_SORT_DECREASING = 2, OR_PLAN_COST_SUMSQ = 4, OR_PLAN_ZIGZAG_CARRY = 8,
       OR_PLAN_AUTO_K = 16 };
enum { SLOT_FREE = 0, SLOT_REGISTERED = 1, SLOT_READY = 2 };

#define TEXT_PAGE_BYTES 4096u /* reading: token ids live in 4 KiB text pages */
#define TEXT_PAGE_IDS 1024u

typedef struct {
  uint64_t page_bytes;
  uint64_t hbm_pages, host_pages;
  uint64_t max_text_tokens;
  uint64_t ring_seed, bind_seed;
  uint64_t gva_hbm_start, gva_host_start, max_size;
  uint32_t hidden;
  uint32_t max_samples, max_spans_per_sample, max_pages_per_span, max_seq_len;
  int32_t placeholder_id;
  uint32_t ring_order, bind_order;
  uint32_t world_size, rank;
  uint64_t max_imported_pages; /* a capacity knob of the device library; unused here */
} oracle_pool_config;

typedef struct {
  uint64_t coef_A, coef_B;
  uint32_t budget_L, n_buckets_K, n_ranks_N, flags;
} oracle_plan_config;

typedef struct {
  uint32_t pos_start, n_tokens;
  uint32_t n_pages; /* 0 until written */
  uint64_t* pages;  /* page GVAs, by ordinal */
  uint32_t grid[3]; /* (T, H, W) of the span's token grid; all zero = none given */
} or_span;

typedef struct {
  int state;
  int remote; /* imported from another process: its pages and text pages are not ours to recycle */
  uint32_t seq_len, n_spans, spans_written;
  uint64_t generation;
  or_span* spans;
  uint32_t n_text_pages;
  uint64_t* text_pages; /* text-page GVAs */
} or_sample;

/* one process's binding as this process holds it (Sec. 3.2: the collected page tables) */
typedef struct {
  int present;
  uint64_t hbm_pages, host_pages, text_pages;
  uint64_t* bind_hbm;  /* vpn -> frame */
  uint64_t* bind_host;
  uint8_t *hbm_mem, *host_mem, *text_mem; /* where this process reaches that process's frames */
} or_peer;

typedef struct oracle_pool {
  oracle_pool_config c;
  or_peer* peers; /* [world_size]; entry c.rank is this process's own binding */
  uint64_t P;        /* hbm_pages + host_pages */
  uint8_t* hbm_mem;  /* backing frames, HBM tier */
  uint8_t* host_mem; /* backing frames, DRAM tier */
  uint8_t* text_mem; /* backing frames, text pages */
  uint64_t* bind_hbm;  /* vpn -> frame */
  uint64_t* bind_host; /* vpn -> frame */
  /* FIFO ring of global page indices */
  uint32_t* ring;
  uint64_t ring_head, ring_count;
  uint64_t n_text_pages;
  uint32_t* tring;
  uint64_t tring_head, tring_count;
  or_sample* samples;
  /* samples in the order in which they became ready (slot, generation) */
  uint32_t* rq_slot; uint64_t* rq_gen; uint64_t rq_head, rq_tail, rq_cap;
  /* first asynchronous ("device-side") error: smallest (call, code, detail) */
  uint64_t call_seq;
  uint64_t status_key; /* UINT64_MAX = none */
} oracle_pool;

typedef struct oracle_plan {
  oracle_plan_config c;
  uint32_t n, n_mb;
  uint32_t* slots;           /* [n] the caller's order */
  uint64_t* slot_generation; /* [n] */
  uint32_t* sample_len;      /* [n] */
  uint64_t* sample_cost;     /* [n] */
  uint32_t* sample_mb;       /* [n] */
  uint32_t* mb_sample_off;   /* [n_mb+1] */
  uint32_t* mb_samples;      /* [n] slots, microbatch-major, append order */
  uint32_t* mb_tokens;       /* [n_mb] */
  uint32_t* mb_lmax;         /* [n_mb] */
  uint32_t* mb_residual;     /* [n_mb] */
  uint64_t* mb_cost;         /* [n_mb] */
  uint32_t* mb_bucket;       /* [n_mb] */
  uint32_t* mb_rank;         /* [n_mb] */
  uint32_t* rank_mb_off;     /* [N+1] */
  uint32_t* rank_mbs;        /* [n_mb] dispatch order per rank */
} oracle_plan;

/* ------------------------------------------------------------------------
 * Counter-based integer hash used for the seeded ring shuffle and the seeded
 * vpn->frame permutation (both sides implement the same published mixer).
 * ---------------------------------------------------------------------- */
static uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
static uint64_t hash2(uint64_t seed, uint64_t i) { return mix64(seed ^ mix64(i)); }

/* Fisher-Yates, i = n-1 .. 1, j = hash(seed, i) mod (i+1). */
static void shuffle_u64(uint64_t* a, uint64_t n, uint64_t seed) {
  for (uint64_t i = n; i-- > 1;) {
    uint64_t j = hash2(seed, i) % (i + 1);
    uint64_t t = a[i]; a[i] = a[j]; a[j] = t;
  }
}
static void shuffle_u32(uint32_t* a, uint64_t n, uint64_t seed) {
  for (uint64_t i = n; i-- > 1;) {
    uint64_t j = hash2(seed, i) % (i + 1);
    uint32_t t = a[i]; a[i] = a[j]; a[j] = t;
  }
}

/* ------------------------------------------------------------------------
 * G. GVA layout and translation (Sec. 3.2).
 * Region t = [start_t, start_t + world_size*max_size); process i owns
 * [start_t + i*max_size, start_t + (i+1)*max_size).  reading: half-open
 * everywhere; defaults start_HBM = 2^44, start_DRAM = 2^45, max_size = 2^40
 * (constants: parity unpinned, the paper gives none).  Page k of tier t of
 * process i has GVA start_t + i*max_size + k*page_bytes; reading: the page
 * table has one entry per pool page.  Text pages follow the embedding pages
 * inside the HBM segment.
 * ---------------------------------------------------------------------- */
uint64_t oracle_segment_base(const oracle_pool* p, uint32_t tier, uint32_t proc) {
  uint64_t start = tier == 0 ? p->c.gva_hbm_start : p->c.gva_host_start;
  return start + (uint64_t)proc * p->c.max_size;
}

uint64_t oracle_page_gva(const oracle_pool* p, uint64_t global_page) {
  if (global_page < p->c.hbm_pages)
    return oracle_segment_base(p, 0, p->c.rank) + global_page * p->c.page_bytes;
  return oracle_segment_base(p, 1, p->c.rank) + (global_page - p->c.hbm_pages) * p->c.page_bytes;
}

/* inverse of oracle_page_gva for a page-aligned GVA of this process */
static uint64_t global_page_of_gva(const oracle_pool* p, uint64_t g) {
  uint64_t host_base = oracle_segment_base(p, 1, p->c.rank);
  if (g >= host_base && g < host_base + p->c.max_size) return p->c.hbm_pages + (g - host_base) / p->c.page_bytes;
  return (g - oracle_segment_base(p, 0, p->c.rank)) / p->c.page_bytes;
}

static uint64_t text_page_gva(const oracle_pool* p, uint64_t k) {
  return oracle_segment_base(p, 0, p->c.rank) + p->c.hbm_pages * p->c.page_bytes + k * TEXT_PAGE_BYTES;
}

/* kind: 0 = HBM embedding page, 1 = DRAM embedding page, 2 = text page; proc = owning process.
 * Translation is local: the region by interval test, the process by division, then that process's table
 * (its own, or one installed by oracle_pool_import_mapping; unknown processes do not translate). */
int32_t oracle_translate_ex(const oracle_pool* p, uint64_t g, uint32_t* proc, uint32_t* kind, uint64_t* frame,
                            uint64_t* offset) {
  const uint64_t W = p->c.world_size, M = p->c.max_size, PS = p->c.page_bytes;
  for (uint32_t t = 0; t < 2; ++t) {
    uint64_t start = t == 0 ? p->c.gva_hbm_start : p->c.gva_host_start;
    if (g < start || g >= start + W * M) continue;
    uint64_t i = (g - start) / M, o = (g - start) % M;
    const or_peer* pr = &p->peers[i];
    if (!pr->present) return OR_ERR_BAD_GVA;
    uint64_t pages = t == 0 ? pr->hbm_pages : pr->host_pages;
    *proc = (uint32_t)i;
    if (o < pages * PS) {
      uint64_t vpn = o / PS;
      *kind = t;
      *frame = t == 0 ? pr->bind_hbm[vpn] : pr->bind_host[vpn];
      *offset = o % PS;
      return OR_OK;
    }
    if (t == 0) {
      uint64_t ot = o - pages * PS;
      if (ot < pr->text_pages * (uint64_t)TEXT_PAGE_BYTES) {
        *kind = 2; *frame = ot / TEXT_PAGE_BYTES; *offset = ot % TEXT_PAGE_BYTES;
        return OR_OK;
      }
    }
    return OR_ERR_BAD_GVA;
  }
  return OR_ERR_BAD_GVA;
}

int32_t oracle_translate(const oracle_pool* p, uint64_t g, uint32_t* kind, uint64_t* frame, uint64_t* offset) {
  uint32_t proc;
  return oracle_translate_ex(p, g, &proc, kind, frame, offset);
}

static uint8_t* resolve(oracle_pool* p, uint64_t g) {
  uint32_t proc, kind; uint64_t frame, off;
  if (oracle_translate_ex(p, g, &proc, &kind, &frame, &off) != OR_OK) return NULL;
  const or_peer* pr = &p->peers[proc];
  if (kind == 0) return pr->hbm_mem + frame * p->c.page_bytes + off;
  if (kind == 1) return pr->host_mem + frame * p->c.page_bytes + off;
  return pr->text_mem + frame * TEXT_PAGE_BYTES + off;
}

/* Sec. 3.1: the scheduler acts once enough paired embeddings have accumulated: a FIFO of samples in the order in
 * which they became ready (reading: completion order; the watermark is a token count chosen by the caller). */
static void ready_push(oracle_pool* p, uint32_t slot) {
  if (p->rq_tail == p->rq_cap) {
    p->rq_cap = p->rq_cap ? 2 * p->rq_cap : 64;
    p->rq_slot = (uint32_t*)realloc(p->rq_slot, p->rq_cap * sizeof(uint32_t));
    p->rq_gen = (uint64_t*)realloc(p->rq_gen, p->rq_cap * sizeof(uint64_t));
  }
  p->rq_slot[p->rq_tail] = slot; p->rq_gen[p->rq_tail] = p->samples[slot].generation; p->rq_tail++;
}

static void note_async_error(oracle_pool* p, int32_t code, uint32_t detail) {
  uint64_t key = (p->call_seq << 40) | ((uint64_t)(uint32_t)(-code) << 32) | detail;
  if (key < p->status_key) p->status_key = key;
}

static uint64_t pages_for_tokens(const oracle_pool* p, uint64_t n_tokens) {
  uint64_t bytes = n_tokens * 2ull * p->c.hidden;
  return (bytes + p->c.page_bytes - 1) / p->c.page_bytes;
}

/* ------------------------------------------------------------------------
 * Pool creation: lay out the regions, bind frames, fill the free rings.
 * ---------------------------------------------------------------------- */
int32_t oracle_pool_create(const oracle_pool_config* cfg, oracle_pool** out) {
  if (!cfg || !out) return OR_ERR_INVALID_ARG;
  oracle_pool_config c = *cfg;
  if (c.gva_hbm_start == 0) c.gva_hbm_start = 1ull << 44;
  if (c.gva_host_start == 0) c.gva_host_start = 1ull << 45;
  if (c.max_size == 0) c.max_size = 1ull << 40;
  if (c.world_size == 0) c.world_size = 1;
  uint64_t PS = c.page_bytes;
  if (PS < 4096 || PS > (2u << 20) || (PS & (PS - 1))) return OR_ERR_INVALID_ARG;
  if (c.hidden == 0 || c.hidden % 8) return OR_ERR_INVALID_ARG;
  if (c.hbm_pages + c.host_pages == 0) return OR_ERR_INVALID_ARG;
  if (c.hbm_pages + c.host_pages > 0xFFFFFFFFull) return OR_ERR_INVALID_ARG;
  if (c.rank >= c.world_size) return OR_ERR_INVALID_ARG;
  if (c.max_samples == 0 || c.max_seq_len == 0) return OR_ERR_INVALID_ARG;
  uint64_t n_text_pages = (c.max_text_tokens + TEXT_PAGE_IDS - 1) / TEXT_PAGE_IDS;
  if (c.hbm_pages * PS + n_text_pages * TEXT_PAGE_BYTES > c.max_size) return OR_ERR_INVALID_ARG;
  if (c.host_pages * PS > c.max_size) return OR_ERR_INVALID_ARG;
  uint64_t span = (uint64_t)c.world_size * c.max_size;
  if (c.gva_hbm_start + span < c.gva_hbm_start || c.gva_host_start + span < c.gva_host_start)
    return OR_ERR_INVALID_ARG;
  if (c.gva_hbm_start < c.gva_host_start + span && c.gva_host_start < c.gva_hbm_start + span)
    return OR_ERR_INVALID_ARG; /* regions overlap */

  oracle_pool* p = (oracle_pool*)calloc(1, sizeof(*p));
  p->c = c;
  p->P = c.hbm_pages + c.host_pages;
  p->n_text_pages = n_text_pages;
  p->hbm_mem = (uint8_t*)malloc(c.hbm_pages * PS + 1);
  p->host_mem = (uint8_t*)malloc(c.host_pages * PS + 1);
  p->text_mem = (uint8_t*)malloc(n_text_pages * TEXT_PAGE_BYTES + 1);
  /* poison: an unwritten byte shows up as 0xFF in any comparison */
  memset(p->hbm_mem, 0xFF, c.hbm_pages * PS);
  memset(p->host_mem, 0xFF, c.host_pages * PS);
  memset(p->text_mem, 0xFF, n_text_pages * TEXT_PAGE_BYTES);

  /* binding: physical memory need not be contiguous; identity, or a seeded
   * permutation per tier (reading; makes the table non-trivial) */
  p->bind_hbm = (uint64_t*)malloc((c.hbm_pages + 1) * sizeof(uint64_t));
  p->bind_host = (uint64_t*)malloc((c.host_pages + 1) * sizeof(uint64_t));
  for (uint64_t k = 0; k < c.hbm_pages; ++k) p->bind_hbm[k] = k;
  for (uint64_t k = 0; k < c.host_pages; ++k) p->bind_host[k] = k;
  if (c.bind_order == OR_BIND_PERMUTED) {
    shuffle_u64(p->bind_hbm, c.hbm_pages, c.bind_seed);
    shuffle_u64(p->bind_host, c.host_pages, c.bind_seed + 1);
  }

  /* free ring over global page indices (parity unpinned: any assignment of
   * free pages would be correct; this one is fixed so results are comparable) */
  p->ring = (uint32_t*)malloc((p->P + 1) * sizeof(uint32_t));
  for (uint64_t k = 0; k < p->P; ++k) p->ring[k] = (uint32_t)k;
  if (c.ring_order == OR_RING_SHUFFLED) shuffle_u32(p->ring, p->P, c.ring_seed);
  p->ring_head = 0; p->ring_count = p->P;

  p->tring = (uint32_t*)malloc((n_text_pages + 1) * sizeof(uint32_t));
  for (uint64_t k = 0; k < n_text_pages; ++k) p->tring[k] = (uint32_t)k;
  p->tring_head = 0; p->tring_count = n_text_pages;

  p->samples = (or_sample*)calloc(c.max_samples, sizeof(or_sample));
  p->status_key = UINT64_MAX;
  p->peers = (or_peer*)calloc(c.world_size, sizeof(or_peer));
  or_peer* self = &p->peers[c.rank];
  self->present = 1;
  self->hbm_pages = c.hbm_pages; self->host_pages = c.host_pages; self->text_pages = n_text_pages;
  self->bind_hbm = p->bind_hbm; self->bind_host = p->bind_host;
  self->hbm_mem = p->hbm_mem; self->host_mem = p->host_mem; self->text_mem = p->text_mem;
  *out = p;
  return OR_OK;
}

static void release_sample_storage(or_sample* s) {
  if (s->spans) {
    for (uint32_t i = 0; i < s->n_spans; ++i) free(s->spans[i].pages);
    free(s->spans);
  }
  free(s->text_pages);
  s->spans = NULL; s->text_pages = NULL;
}

int32_t oracle_pool_destroy(oracle_pool* p) {
  if (!p) return OR_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < p->c.max_samples; ++i) release_sample_storage(&p->samples[i]);
  for (uint32_t i = 0; i < p->c.world_size; ++i)
    if (i != p->c.rank && p->peers[i].present) { free(p->peers[i].bind_hbm); free(p->peers[i].bind_host); }
  free(p->peers); free(p->rq_slot); free(p->rq_gen);
  free(p->samples); free(p->ring); free(p->tring); free(p->bind_hbm); free(p->bind_host);
  free(p->hbm_mem); free(p->host_mem); free(p->text_mem); free(p);
  return OR_OK;
}

/* ------------------------------------------------------------------------
 * T. Register samples: text tokens and pairing metadata (Sec. 3.1: text
 * tokens go into the same pool, lightweight metadata tracks the pairing).
 * reading: a sample is input_ids[seq_len] in which span i occupies one run of
 * placeholder ids starting at span_pos[i], n_tokens[i] long; runs sorted and
 * non-overlapping.  All checks first, then the effect (all-or-nothing).
 * ---------------------------------------------------------------------- */
int32_t oracle_pool_register_samples(oracle_pool* p, uint32_t n, const uint32_t* slot,
                                     const uint32_t* seq_len, const uint32_t* n_spans,
                                     const uint32_t* span_pos, const uint32_t* span_tokens,
                                     const int32_t* input_ids) {
  if (!p) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (n == 0) return OR_OK;
  if (!slot || !seq_len || !n_spans || !input_ids) return OR_ERR_INVALID_ARG;
  uint64_t text_need = 0, sp = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= p->c.max_samples) return OR_ERR_INVALID_ARG;
    if (p->samples[slot[i]].state != SLOT_FREE) return OR_ERR_SLOT_IN_USE;
    for (uint32_t j = 0; j < i; ++j)
      if (slot[j] == slot[i]) return OR_ERR_SLOT_IN_USE;
    if (seq_len[i] == 0) return OR_ERR_INVALID_ARG;
    if (seq_len[i] > p->c.max_seq_len) return OR_ERR_CAPACITY;
    if (n_spans[i] > p->c.max_spans_per_sample) return OR_ERR_CAPACITY;
    if (n_spans[i] && (!span_pos || !span_tokens)) return OR_ERR_INVALID_ARG;
    uint64_t prev_end = 0;
    for (uint32_t j = 0; j < n_spans[i]; ++j, ++sp) {
      if (span_tokens[sp] == 0) return OR_ERR_INVALID_ARG;
      if ((uint64_t)span_pos[sp] + span_tokens[sp] > seq_len[i]) return OR_ERR_INVALID_ARG;
      if (span_pos[sp] < prev_end) return OR_ERR_INVALID_ARG;
      prev_end = (uint64_t)span_pos[sp] + span_tokens[sp];
      if (pages_for_tokens(p, span_tokens[sp]) > p->c.max_pages_per_span) return OR_ERR_CAPACITY;
    }
    text_need += (seq_len[i] + TEXT_PAGE_IDS - 1) / TEXT_PAGE_IDS;
  }
  if (text_need > p->tring_count) return OR_ERR_CAPACITY;

  sp = 0;
  uint64_t idoff = 0;
  for (uint32_t i = 0; i < n; ++i) {
    or_sample* s = &p->samples[slot[i]];
    s->state = n_spans[i] == 0 ? SLOT_READY : SLOT_REGISTERED; /* text-only: paired at once */
    if (s->state == SLOT_READY) ready_push(p, slot[i]);
    s->seq_len = seq_len[i]; s->n_spans = n_spans[i]; s->spans_written = 0; s->remote = 0;
    s->spans = (or_span*)calloc(n_spans[i] + 1, sizeof(or_span));
    uint64_t placeholders = 0;
    int bad = 0;
    for (uint32_t j = 0; j < n_spans[i]; ++j, ++sp) {
      s->spans[j].pos_start = span_pos[sp];
      s->spans[j].n_tokens = span_tokens[sp];
      placeholders += span_tokens[sp];
      for (uint32_t t = 0; t < span_tokens[sp]; ++t)
        if (input_ids[idoff + span_pos[sp] + t] != p->c.placeholder_id) bad = 1;
    }
    uint64_t seen = 0;
    for (uint32_t t = 0; t < seq_len[i]; ++t)
      if (input_ids[idoff + t] == p->c.placeholder_id) ++seen;
    if (seen != placeholders) bad = 1; /* stray placeholder outside every run */
    if (bad) note_async_error(p, OR_ERR_PLACEHOLDER_MISMATCH, slot[i]);
    /* ids into text pages popped from the text ring, page by page */
    s->n_text_pages = (seq_len[i] + TEXT_PAGE_IDS - 1) / TEXT_PAGE_IDS;
    s->text_pages = (uint64_t*)malloc(s->n_text_pages * sizeof(uint64_t));
    for (uint32_t k = 0; k < s->n_text_pages; ++k) {
      uint32_t tp = p->tring[p->tring_head];
      p->tring_head = (p->tring_head + 1) % p->n_text_pages; p->tring_count--;
      s->text_pages[k] = text_page_gva(p, tp);
    }
    for (uint32_t t = 0; t < seq_len[i]; ++t) {
      uint8_t* dst = resolve(p, s->text_pages[t / TEXT_PAGE_IDS] + (uint64_t)(t % TEXT_PAGE_IDS) * 4);
      memcpy(dst, &input_ids[idoff + t], 4);
    }
    idoff += seq_len[i];
  }
  return OR_OK;
}

/* ------------------------------------------------------------------------
 * W. fp32 -> bf16, IEEE round-to-nearest-even on the bit pattern; denormals
 * kept; overflow rounds to +-Inf.  reading (parity unpinned): every NaN
 * becomes the sign-preserving quiet NaN 0x7FC0 / 0xFFC0.
 * ---------------------------------------------------------------------- */
uint16_t oracle_f32_to_bf16_rne(uint32_t u) {
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)(((u >> 16) & 0x8000u) | 0x7FC0u);
  return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);
}

/* ------------------------------------------------------------------------
 * F + W. Producer write (Sec. 3.1, 3.2: encoders place embeddings into their
 * own segment of the pool).  Page allocation: span q of the call takes the
 * next ceil(n_tokens*2H / page_bytes) entries from the ring head, spans in
 * argument order; whole pages per span.  Byte b of the span's bf16 row-major
 * [n_tokens, H] image lives in page b / page_bytes at offset b % page_bytes;
 * the tail of the last page keeps whatever it held.
 * ---------------------------------------------------------------------- */
int32_t oracle_pool_write_embeddings(oracle_pool* p, uint32_t n_spans, const uint32_t* slot,
                                     const uint32_t* span_idx, const uint32_t* n_tokens,
                                     const void* const* src, uint32_t src_dtype) {
  if (!p) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (src_dtype != OR_BF16 && src_dtype != OR_F32) return OR_ERR_INVALID_ARG;
  if (n_spans == 0) return OR_OK;
  if (!slot || !span_idx || !n_tokens || !src) return OR_ERR_INVALID_ARG;
  uint64_t need = 0;
  for (uint32_t q = 0; q < n_spans; ++q) {
    if (slot[q] >= p->c.max_samples) return OR_ERR_INVALID_ARG;
    or_sample* s = &p->samples[slot[q]];
    if (s->state == SLOT_FREE) return OR_ERR_UNKNOWN_SAMPLE;
    if (span_idx[q] >= s->n_spans) return OR_ERR_INVALID_ARG;
    if (n_tokens[q] != s->spans[span_idx[q]].n_tokens) return OR_ERR_INVALID_ARG;
    if (!src[q]) return OR_ERR_INVALID_ARG;
    if (s->spans[span_idx[q]].n_pages != 0) return OR_ERR_ALREADY_WRITTEN;
    for (uint32_t r = 0; r < q; ++r)
      if (slot[r] == slot[q] && span_idx[r] == span_idx[q]) return OR_ERR_ALREADY_WRITTEN;
    need += pages_for_tokens(p, n_tokens[q]);
  }
  if (need > p->ring_count) return OR_ERR_POOL_EXHAUSTED;

  const uint64_t PS = p->c.page_bytes, H = p->c.hidden;
  for (uint32_t q = 0; q < n_spans; ++q) {
    or_sample* s = &p->samples[slot[q]];
    or_span* sp = &s->spans[span_idx[q]];
    uint64_t k = pages_for_tokens(p, n_tokens[q]);
    sp->n_pages = (uint32_t)k;
    sp->pages = (uint64_t*)malloc(k * sizeof(uint64_t));
    for (uint64_t o = 0; o < k; ++o) {
      uint32_t g = p->ring[p->ring_head];
      p->ring_head = (p->ring_head + 1) % p->P; p->ring_count--;
      sp->pages[o] = oracle_page_gva(p, g);
    }
    uint64_t n_bytes = (uint64_t)n_tokens[q] * H * 2, b = 0;
    while (b < n_bytes) { /* maximal run inside one page (page_bytes is even: no element straddles) */
      uint64_t off = b % PS;
      uint64_t run = PS - off < n_bytes - b ? PS - off : n_bytes - b;
      uint8_t* dst = resolve(p, sp->pages[b / PS] + off);
      if (src_dtype == OR_BF16) {
        memcpy(dst, (const uint8_t*)src[q] + b, run);
      } else {
        for (uint64_t e = 0; e < run / 2; ++e) {
          uint16_t v = oracle_f32_to_bf16_rne(((const uint32_t*)src[q])[b / 2 + e]);
          memcpy(dst + 2 * e, &v, 2);
        }
      }
      b += run;
    }
    s->spans_written++;
    if (s->spans_written == s->n_spans) { s->state = SLOT_READY; ready_push(p, slot[q]); } /* "paired" */
  }
  return OR_OK;
}

/* ------------------------------------------------------------------------
 * F. Free: samples in argument order, spans by index, pages by ordinal, each
 * pushed to the ring tail; the slot returns to FREE.
 * ---------------------------------------------------------------------- */
int32_t oracle_pool_free(oracle_pool* p, const uint32_t* slot, uint32_t n) {
  if (!p) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (n == 0) return OR_OK;
  if (!slot) return OR_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= p->c.max_samples) return OR_ERR_INVALID_ARG;
    if (p->samples[slot[i]].state == SLOT_FREE) return OR_ERR_UNKNOWN_SAMPLE;
    for (uint32_t j = 0; j < i; ++j)
      if (slot[j] == slot[i]) return OR_ERR_UNKNOWN_SAMPLE;
  }
  for (uint32_t i = 0; i < n; ++i) {
    or_sample* s = &p->samples[slot[i]];
    if (!s->remote) { /* an imported sample's pages and text pages belong to the process that wrote them */
      for (uint32_t j = 0; j < s->n_spans; ++j)
        for (uint32_t o = 0; o < s->spans[j].n_pages; ++o) {
          uint64_t idx = global_page_of_gva(p, s->spans[j].pages[o]);
          p->ring[(p->ring_head + p->ring_count) % p->P] = (uint32_t)idx;
          p->ring_count++;
        }
      for (uint32_t k = 0; k < s->n_text_pages; ++k) {
        uint64_t tp = (s->text_pages[k] - text_page_gva(p, 0)) / TEXT_PAGE_BYTES;
        p->tring[(p->tring_head + p->tring_count) % p->n_text_pages] = (uint32_t)tp;
        p->tring_count++;
      }
    }
    release_sample_storage(s);
    s->state = SLOT_FREE; s->n_spans = 0; s->seq_len = 0; s->spans_written = 0; s->n_text_pages = 0; s->remote = 0;
    s->generation++;
  }
  return OR_OK;
}

/* ------------------------------------------------------------------------
 * P. Dynamic packing (Algorithm 1, Eq. 3).
 * ---------------------------------------------------------------------- */

/* Best-fit packing, Algorithm 1 lines 1-11, as the definition the segment
 * tree accelerates: the open microbatch with the smallest residual >= l.
 * reading (tie-break, parity unpinned): among equal residuals, the one whose
 * residual changed most recently.  reading: l_min = the smallest length of
 * this call, so the removal step (lines 10-11) never changes the result and
 * is omitted here; oracle_bestfit_segment_tree below performs it literally. */
static uint32_t best_fit(uint32_t n, const uint32_t* len, uint32_t L, uint32_t* sample_mb,
                         uint32_t* P, uint32_t* tokens, uint32_t* lmax, uint32_t* count) {
  uint32_t n_mb = 0;
  uint32_t* stamp = (uint32_t*)malloc((n + 1) * sizeof(uint32_t));
  for (uint32_t t = 0; t < n; ++t) {
    uint32_t l = len[t];
    int64_t best = -1;
    for (uint32_t j = 0; j < n_mb; ++j) {
      if (P[j] < l) continue;
      if (best < 0 || P[j] < P[best] || (P[j] == P[best] && stamp[j] > stamp[best])) best = j;
    }
    uint32_t j;
    if (best >= 0) {
      j = (uint32_t)best;
      P[j] -= l; tokens[j] += l; if (l > lmax[j]) lmax[j] = l; count[j]++;
    } else {
      j = n_mb++;
      P[j] = L - l; tokens[j] = l; lmax[j] = l; count[j] = 1;
    }
    stamp[j] = t;
    sample_mb[t] = j;
  }
  free(stamp);
  return n_mb;
}

/* Second, literal statement of Algorithm 1 lines 1-11: a segment tree over
 * the residual values [0, L]; leaf r holds the open microbatches whose
 * residual is r (most recently changed on top), an inner node the largest
 * non-empty residual below it; the query prefers the left (smaller) subtree
 * whenever its maximum is >= l; a microbatch whose residual drops below l_min
 * is removed.  Returns n_mb; used by tests to pin best_fit. */
uint32_t oracle_bestfit_segment_tree(uint32_t n, const uint32_t* len, uint32_t L, uint32_t l_min,
                                     uint32_t* sample_mb) {
  uint32_t leaves = 1; while (leaves < L + 1) leaves <<= 1;
  int64_t* node = (int64_t*)malloc(2ull * leaves * sizeof(int64_t));
  for (uint32_t i = 0; i < 2 * leaves; ++i) node[i] = -1;
  int64_t* top = (int64_t*)malloc(((uint64_t)L + 1) * sizeof(int64_t)); /* stack top per residual */
  for (uint32_t r = 0; r <= L; ++r) top[r] = -1;
  int64_t* below = (int64_t*)malloc(((uint64_t)n + 1) * sizeof(int64_t));
  uint32_t* P = (uint32_t*)malloc(((uint64_t)n + 1) * sizeof(uint32_t));
  uint32_t n_mb = 0;
  for (uint32_t t = 0; t < n; ++t) {
    uint32_t l = len[t];
    int64_t j = -1;
    if (node[1] >= (int64_t)l) {
      uint32_t v = 1;
      while (v < leaves) v = node[2 * v] >= (int64_t)l ? 2 * v : 2 * v + 1;
      uint32_t r = v - leaves;
      j = top[r];
      top[r] = below[j]; /* take it off leaf r */
      if (top[r] < 0) { node[v] = -1; for (v >>= 1; v >= 1; v >>= 1) node[v] = node[2*v] > node[2*v+1] ? node[2*v] : node[2*v+1]; }
      P[j] -= l;
    } else {
      j = n_mb++;
      P[j] = L - l;
    }
    sample_mb[t] = (uint32_t)j;
    if (P[j] >= l_min) { /* (re)insert at its new residual unless removed */
      uint32_t r = P[j];
      below[j] = top[r]; top[r] = j;
      uint32_t v = leaves + r; node[v] = r;
      for (v >>= 1; v >= 1; v >>= 1) node[v] = node[2*v] > node[2*v+1] ? node[2*v] : node[2*v+1];
    }
  }
  free(node); free(top); free(below); free(P);
  return n_mb;
}

/* Eq. 3 scaled to integers: A*sum(l) + B*lmax^2; with (A,B) = (L,1) this is
 * L^2 * Cost(B_j) exactly.  The quadratic term is lmax^2, the term Eq. 3 has. */
uint64_t oracle_cost_int(uint64_t A, uint64_t B, uint64_t sum_len, uint64_t lmax) {
  return A * sum_len + B * lmax * lmax;
}

/* Two-dimension load balancing, Algorithm 1 lines 12-27, on given costs.
 * Outputs: bucket[n_mb], rank[n_mb], rank_mb_off[N+1], rank_mbs[n_mb]. */
void oracle_balance(uint32_t n_mb, const uint64_t* cost, uint32_t K, uint32_t N, int carry, uint32_t* bucket,
                    uint32_t* rank, uint32_t* rank_mb_off, uint32_t* rank_mbs) {
  /* lines 12-14: buckets.  reading (parity unpinned): equal-width
   * quantisation of the observed cost range into K buckets. */
  uint64_t lo = UINT64_MAX, hi = 0;
  for (uint32_t j = 0; j < n_mb; ++j) {
    if (cost[j] < lo) lo = cost[j];
    if (cost[j] > hi) hi = cost[j];
  }
  for (uint32_t j = 0; j < n_mb; ++j) {
    /* (cost-lo)*K / (hi-lo+1), in 128-bit so nothing overflows */
    unsigned __int128 num = (unsigned __int128)(cost[j] - lo) * K;
    bucket[j] = (uint32_t)(num / ((unsigned __int128)(hi - lo) + 1));
  }
  /* Algorithm 1 lines 15-27, the deal.  Readings: buckets are taken from the highest to the lowest; inside a
   * bucket the microbatches are ordered by cost, descending, equal costs by index, ascending; the deal of a bucket
   * ends with its list.  Dealing N at a time over Rank_0..Rank_{N-1} and back means that the i-th microbatch of a
   * bucket's ordered list sits at place i mod N of round i div N, and that odd rounds run from the last rank
   * down: rank = i mod N in even rounds, N-1 - (i mod N) in odd rounds; every bucket starts again at round 0 (the
   * algorithm sets its position and direction inside the loop over buckets).
   * Variant `carry`: one continuous zig-zag over the buckets' lists in turn: the position inside the current round
   * and the direction carry over from bucket to bucket. */
  uint32_t* list = (uint32_t*)calloc((size_t)n_mb + 1, sizeof(uint32_t));
  uint32_t* order = (uint32_t*)calloc((size_t)n_mb + 1, sizeof(uint32_t)); /* global dispatch order */
  uint32_t n_order = 0;
  uint32_t r_next = 0; int forward_c = 1; /* carried state: next rank to serve and the direction */
  for (int64_t k = (int64_t)K - 1; k >= 0; --k) {
    uint32_t m = 0;
    for (uint32_t j = 0; j < n_mb; ++j)
      if (bucket[j] == (uint32_t)k) list[m++] = j;
    for (uint32_t i = 1; i < m; ++i) { /* insertion sort: stable, so index order survives ties */
      uint32_t x = list[i]; int64_t h = (int64_t)i - 1;
      while (h >= 0 && cost[list[h]] < cost[x]) { list[h + 1] = list[h]; --h; }
      list[h + 1] = x;
    }
    if (carry) {
      for (uint32_t a = 0; a < m; ++a) {
        rank[list[a]] = r_next; order[n_order++] = list[a];
        if (forward_c) { if (r_next + 1 == N) forward_c = 0; else ++r_next; }   /* R0..R(N-1), then R(N-1)..R0 */
        else           { if (r_next == 0) forward_c = 1; else --r_next; }
      }
      continue;
    }
    for (uint32_t i = 0; i < m; ++i) {
      const uint32_t round = i / N, place = i % N;
      rank[list[i]] = (round & 1u) ? N - 1 - place : place;
      order[n_order++] = list[i];
    }
  }
  /* per-rank lists, in the order the microbatches were dealt */
  rank_mb_off[0] = 0;
  for (uint32_t r = 0; r < N; ++r) {
    rank_mb_off[r + 1] = rank_mb_off[r];
    for (uint32_t i = 0; i < n_order; ++i)
      if (rank[order[i]] == r) rank_mbs[rank_mb_off[r + 1]++] = order[i];
  }
  free(list); free(order);
}

/* argument check: the largest cost a microbatch can have, A*L + B*L^2, must fit 64 bits */
static int cost_fits(const oracle_plan_config* cfg) {
  unsigned __int128 mx = (unsigned __int128)cfg->coef_A * cfg->budget_L +
                         (unsigned __int128)cfg->coef_B * cfg->budget_L * cfg->budget_L;
  return (mx >> 64) == 0;
}

void oracle_plan_destroy_inner(oracle_plan* pl) {
  free(pl->slots); free(pl->slot_generation); free(pl->sample_len); free(pl->sample_cost);
  free(pl->sample_mb); free(pl->mb_sample_off); free(pl->mb_samples); free(pl->mb_tokens);
  free(pl->mb_lmax); free(pl->mb_residual); free(pl->mb_cost); free(pl->mb_bucket);
  free(pl->mb_rank); free(pl->rank_mb_off); free(pl->rank_mbs);
}
int32_t oracle_plan_destroy(oracle_plan* pl) {
  if (!pl) return OR_ERR_INVALID_ARG;
  oracle_plan_destroy_inner(pl); free(pl);
  return OR_OK;
}

/* Packing + load balancing over explicit lengths (no pool needed): the whole
 * of Algorithm 1.  slots may be NULL (then sample t is "slot" t). */
int32_t oracle_plan_from_lengths(const uint32_t* slots, const uint32_t* len, uint32_t n,
                                 const oracle_plan_config* cfg, oracle_plan** out) {
  if (!cfg || !out) return OR_ERR_INVALID_ARG;
  const uint32_t L = cfg->budget_L, K = cfg->n_buckets_K, N = cfg->n_ranks_N;
  if (L == 0 || K == 0 || N == 0) return OR_ERR_INVALID_ARG;
  if (!cost_fits(cfg)) return OR_ERR_INVALID_ARG;
  for (uint32_t t = 0; t < n; ++t) {
    if (len[t] == 0) return OR_ERR_INVALID_ARG;
    if (len[t] > L) return OR_ERR_TOO_LONG;
  }
  oracle_plan* pl = (oracle_plan*)calloc(1, sizeof(*pl));
  pl->c = *cfg; pl->n = n;
#define ALLOC(T, cnt) (T*)calloc((size_t)(cnt) + 1, sizeof(T))
  pl->slots = ALLOC(uint32_t, n); pl->slot_generation = ALLOC(uint64_t, n);
  pl->sample_len = ALLOC(uint32_t, n); pl->sample_cost = ALLOC(uint64_t, n);
  pl->sample_mb = ALLOC(uint32_t, n); pl->mb_samples = ALLOC(uint32_t, n);
  pl->mb_sample_off = ALLOC(uint32_t, n + 1);
  pl->mb_tokens = ALLOC(uint32_t, n); pl->mb_lmax = ALLOC(uint32_t, n);
  pl->mb_residual = ALLOC(uint32_t, n); pl->mb_cost = ALLOC(uint64_t, n);
  pl->mb_bucket = ALLOC(uint32_t, n); pl->mb_rank = ALLOC(uint32_t, n);
  pl->rank_mb_off = ALLOC(uint32_t, N + 1); pl->rank_mbs = ALLOC(uint32_t, n);
  uint32_t* count = ALLOC(uint32_t, n);
  for (uint32_t t = 0; t < n; ++t) {
    pl->slots[t] = slots ? slots[t] : t;
    pl->sample_len[t] = len[t];
    /* per-sample score: Eq. 3 on a singleton microbatch */
    pl->sample_cost[t] = oracle_cost_int(cfg->coef_A, cfg->coef_B, len[t], len[t]);
  }
  /* packing order: the caller's order (reading), or, as a variant, longest first (best-fit decreasing;
   * equal lengths keep the caller's order) */
  uint32_t* ord = ALLOC(uint32_t, n);
  uint32_t* olen = ALLOC(uint32_t, n);
  uint32_t* omb = ALLOC(uint32_t, n);
  for (uint32_t t = 0; t < n; ++t) ord[t] = t;
  if (cfg->flags & OR_PLAN_SORT_DECREASING)
    for (uint32_t i = 1; i < n; ++i) { /* stable insertion sort by length, descending */
      uint32_t x = ord[i]; int64_t h = (int64_t)i - 1;
      while (h >= 0 && len[ord[h]] < len[x]) { ord[h + 1] = ord[h]; --h; }
      ord[h + 1] = x;
    }
  for (uint32_t r = 0; r < n; ++r) olen[r] = len[ord[r]];
  /* lines 1-11 */
  uint32_t n_mb = best_fit(n, olen, L, omb, pl->mb_residual, pl->mb_tokens, pl->mb_lmax, count);
  pl->n_mb = n_mb;
  for (uint32_t r = 0; r < n; ++r) pl->sample_mb[ord[r]] = omb[r];
  /* samples inside a microbatch stay in packing order (line 5: append) */
  for (uint32_t j = 0; j < n_mb; ++j) pl->mb_sample_off[j + 1] = pl->mb_sample_off[j] + count[j];
  for (uint32_t j = 0; j < n_mb; ++j) {
    uint32_t w = pl->mb_sample_off[j];
    for (uint32_t r = 0; r < n; ++r)
      if (omb[r] == j) pl->mb_samples[w++] = pl->slots[ord[r]];
  }
  /* lines 12-14: Cost(B_j).  As printed the quadratic term is lmax^2; variant: the sum of squares */
  for (uint32_t j = 0; j < n_mb; ++j) {
    if (cfg->flags & OR_PLAN_COST_SUMSQ) {
      uint64_t sq = 0;
      for (uint32_t r = 0; r < n; ++r)
        if (omb[r] == j) sq += (uint64_t)olen[r] * olen[r];
      pl->mb_cost[j] = cfg->coef_A * pl->mb_tokens[j] + cfg->coef_B * sq;
    } else {
      pl->mb_cost[j] = oracle_cost_int(cfg->coef_A, cfg->coef_B, pl->mb_tokens[j], pl->mb_lmax[j]);
    }
  }
  /* lines 12-27: buckets and zig-zag dispatch.  The paper does not say how many clusters there are.
   * Default: the caller's K.  Variant AUTO_K: as many buckets as there are full zig-zag round trips
   * (one forward and one backward pass over the N ranks = 2N microbatches), at least 1, at most the caller's K,
   * so that every bucket can pair high and low costs on each rank. */
  uint32_t K_used = K;
  if (cfg->flags & OR_PLAN_AUTO_K) {
    uint64_t trips = ((uint64_t)n_mb + 2ull * N - 1) / (2ull * N);
    if (trips < 1) trips = 1;
    if (trips < K_used) K_used = (uint32_t)trips;
  }
  oracle_balance(n_mb, pl->mb_cost, K_used, N, (cfg->flags & OR_PLAN_ZIGZAG_CARRY) != 0, pl->mb_bucket, pl->mb_rank,
                 pl->rank_mb_off, pl->rank_mbs);
  free(ord); free(olen); free(omb);
  free(count);
  *out = pl;
  return OR_OK;
}

int32_t oracle_pool_plan_microbatches(oracle_pool* p, const uint32_t* slots, uint32_t n,
                                      const oracle_plan_config* cfg, oracle_plan** out) {
  if (!p || !cfg || !out) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (cfg->budget_L == 0 || cfg->n_buckets_K == 0 || cfg->n_ranks_N == 0) return OR_ERR_INVALID_ARG;
  if (!cost_fits(cfg)) return OR_ERR_INVALID_ARG;
  if (n && !slots) return OR_ERR_INVALID_ARG;
  uint32_t* len = (uint32_t*)calloc((size_t)n + 1, sizeof(uint32_t));
  uint8_t* seen = (uint8_t*)calloc(p->c.max_samples, 1);
  int32_t rc = OR_OK;
  for (uint32_t t = 0; t < n && rc == OR_OK; ++t) {
    if (slots[t] >= p->c.max_samples) { rc = OR_ERR_INVALID_ARG; break; }
    or_sample* s = &p->samples[slots[t]];
    if (s->state == SLOT_FREE) rc = OR_ERR_UNKNOWN_SAMPLE;
    else if (seen[slots[t]]) rc = OR_ERR_INVALID_ARG;
    else if (s->state != SLOT_READY && !(cfg->flags & OR_PLAN_ALLOW_UNWRITTEN)) rc = OR_ERR_NOT_READY;
    else if (s->seq_len > cfg->budget_L) rc = OR_ERR_TOO_LONG;
    seen[slots[t]] = 1;
    len[t] = s->seq_len; /* l(s): the LLM-side length, text + all vision tokens */
  }
  if (rc == OR_OK) rc = oracle_plan_from_lengths(slots, len, n, cfg, out);
  if (rc == OR_OK)
    for (uint32_t t = 0; t < n; ++t) (*out)->slot_generation[t] = p->samples[slots[t]].generation;
  free(len); free(seen);
  return rc;
}

/* ------------------------------------------------------------------------
 * A. Packed assembly (Sec. 3.1-3.2: the backbone consumes microbatches by
 * GVA; Sec. 4.1: image and text subsequences are interleaved).
 * Output row cu_seqlens[q] + p of a microbatch = row (p - pos_start) of the
 * span whose placeholder run contains p, read through the span's page list
 * and the page table; otherwise embed_table[input_ids[p]].  position id = p.
 * ---------------------------------------------------------------------- */
int32_t oracle_pool_gather_packed(oracle_pool* p, const oracle_plan* pl, uint32_t mb_begin,
                                  uint32_t mb_end, const void* embed_table, uint32_t vocab,
                                  void* out_embeds, int32_t* out_cu_seqlens,
                                  int32_t* out_position_ids) {
  if (!p || !pl) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (mb_begin > mb_end || mb_end > pl->n_mb) return OR_ERR_INVALID_ARG;
  for (uint32_t t = 0; t < pl->n; ++t) {
    or_sample* s = &p->samples[pl->slots[t]];
    if (s->state != SLOT_READY || s->generation != pl->slot_generation[t]) return OR_ERR_NOT_READY;
  }
  if (mb_begin == mb_end) return OR_OK;
  if (!embed_table || !out_embeds || !out_cu_seqlens || !out_position_ids) return OR_ERR_INVALID_ARG;
  const uint64_t PS = p->c.page_bytes, row_bytes = 2ull * p->c.hidden;
  uint8_t* out = (uint8_t*)out_embeds;
  uint64_t row = 0, cu_w = 0;
  for (uint32_t j = mb_begin; j < mb_end; ++j) {
    int32_t cu = 0;
    out_cu_seqlens[cu_w++] = 0;
    for (uint32_t qi = pl->mb_sample_off[j]; qi < pl->mb_sample_off[j + 1]; ++qi) {
      or_sample* s = &p->samples[pl->mb_samples[qi]];
      for (uint32_t pos = 0; pos < s->seq_len; ++pos, ++row) {
        int32_t id;
        memcpy(&id, resolve(p, s->text_pages[pos / TEXT_PAGE_IDS] + (uint64_t)(pos % TEXT_PAGE_IDS) * 4), 4);
        out_position_ids[row] = (int32_t)pos;
        const or_span* sp = NULL;
        for (uint32_t i = 0; i < s->n_spans; ++i)
          if (pos >= s->spans[i].pos_start && pos < s->spans[i].pos_start + s->spans[i].n_tokens) sp = &s->spans[i];
        uint8_t* dst = out + row * row_bytes;
        if (sp) {
          uint64_t b = (uint64_t)(pos - sp->pos_start) * row_bytes;
          uint64_t done = 0;
          while (done < row_bytes) { /* maximal run inside one page */
            uint64_t off = (b + done) % PS;
            uint64_t run = PS - off < row_bytes - done ? PS - off : row_bytes - done;
            uint8_t* src = resolve(p, sp->pages[(b + done) / PS] + off);
            if (!src) { note_async_error(p, OR_ERR_BAD_GVA, (uint32_t)row); break; }
            memcpy(dst + done, src, run);
            done += run;
          }
        } else if (id < 0 || (uint32_t)id >= vocab) {
          note_async_error(p, OR_ERR_BAD_TOKEN_ID, (uint32_t)row); /* row left untouched */
        } else {
          memcpy(dst, (const uint8_t*)embed_table + (uint64_t)id * row_bytes, row_bytes);
        }
      }
      cu += (int32_t)s->seq_len;
      out_cu_seqlens[cu_w++] = cu;
    }
  }
  return OR_OK;
}

/* The microbatches named in mb_list, in list order (Algorithm 1 deals microbatches to ranks, lines 15-27: a rank
 * consumes its own list, which is not a contiguous range).  Outputs are the concatenation of what
 * oracle_pool_gather_packed writes for each [j, j+1).  An index may repeat. */
int32_t oracle_pool_gather_list(oracle_pool* p, const oracle_plan* pl, const uint32_t* mb_list, uint32_t n_list,
                                const void* embed_table, uint32_t vocab, void* out_embeds,
                                int32_t* out_cu_seqlens, int32_t* out_position_ids) {
  if (!p || !pl || (n_list && !mb_list)) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  for (uint32_t i = 0; i < n_list; ++i)
    if (mb_list[i] >= pl->n_mb) return OR_ERR_INVALID_ARG;
  for (uint32_t t = 0; t < pl->n; ++t) {
    or_sample* s = &p->samples[pl->slots[t]];
    if (s->state != SLOT_READY || s->generation != pl->slot_generation[t]) return OR_ERR_NOT_READY;
  }
  if (n_list == 0) return OR_OK;
  if (!embed_table || !out_embeds || !out_cu_seqlens || !out_position_ids) return OR_ERR_INVALID_ARG;
  const uint64_t row_bytes = 2ull * p->c.hidden;
  const uint64_t call = p->call_seq;
  uint64_t row = 0, cu_w = 0;
  for (uint32_t i = 0; i < n_list; ++i) {
    const uint32_t j = mb_list[i];
    /* one microbatch through the packed assembly; asynchronous errors keep this call's number and report the row
     * index in the list's output */
    const uint64_t key_before = p->status_key;
    p->status_key = UINT64_MAX;
    int32_t rc = oracle_pool_gather_packed(p, pl, j, j + 1, embed_table, vocab, (uint8_t*)out_embeds + row * row_bytes,
                                           out_cu_seqlens + cu_w, out_position_ids + row);
    p->call_seq = call;
    if (p->status_key != UINT64_MAX) {
      const uint64_t code = (p->status_key >> 32) & 0xFF, detail = (p->status_key & 0xFFFFFFFFull) + row;
      p->status_key = (call << 40) | (code << 32) | detail;
    }
    if (key_before < p->status_key) p->status_key = key_before;
    if (rc != OR_OK) return rc;
    row += pl->mb_tokens[j];
    cu_w += (uint64_t)(pl->mb_sample_off[j + 1] - pl->mb_sample_off[j]) + 1;
  }
  return OR_OK;
}

/* ------------------------------------------------------------------------
 * More than one process (Sec. 3.2): each process exports its memory mapping,
 * the others update their page tables; samples cross processes as descriptors
 * (lengths, spans, page GVAs, text-page GVAs) and are read in place.
 * Blob formats are this file's own.
 * ---------------------------------------------------------------------- */
typedef struct {
  uint64_t magic, page_bytes, hbm_pages, host_pages, text_pages, gva_hbm_start, gva_host_start, max_size;
  uint32_t rank, world_size;
} or_map_header;
#define OR_MAP_MAGIC 0x4F5241434C454D50ull
#define OR_SMP_MAGIC 0x4F5241434C455350ull

int32_t oracle_pool_export_mapping(oracle_pool* p, void* buf, uint64_t cap, uint64_t* bytes) {
  if (!p) return OR_ERR_INVALID_ARG;
  uint64_t need = sizeof(or_map_header) + 8 * (p->c.hbm_pages + p->c.host_pages);
  if (bytes) *bytes = need;
  if (!buf) return OR_OK;
  if (cap < need) return OR_ERR_CAPACITY;
  or_map_header h;
  memset(&h, 0, sizeof(h));
  h.magic = OR_MAP_MAGIC; h.page_bytes = p->c.page_bytes; h.hbm_pages = p->c.hbm_pages; h.host_pages = p->c.host_pages;
  h.text_pages = p->n_text_pages; h.gva_hbm_start = p->c.gva_hbm_start; h.gva_host_start = p->c.gva_host_start;
  h.max_size = p->c.max_size; h.rank = p->c.rank; h.world_size = p->c.world_size;
  memcpy(buf, &h, sizeof(h));
  memcpy((uint8_t*)buf + sizeof(h), p->bind_hbm, 8 * p->c.hbm_pages);
  memcpy((uint8_t*)buf + sizeof(h) + 8 * p->c.hbm_pages, p->bind_host, 8 * p->c.host_pages);
  return OR_OK;
}

/* peer_*: where this process reaches the peer's frames (host pointers here) */
int32_t oracle_pool_import_mapping(oracle_pool* p, const void* buf, uint64_t bytes, void* peer_hbm, void* peer_host,
                                   void* peer_text) {
  if (!p || !buf || bytes < sizeof(or_map_header)) return OR_ERR_INVALID_ARG;
  or_map_header h;
  memcpy(&h, buf, sizeof(h));
  if (h.magic != OR_MAP_MAGIC || bytes != sizeof(h) + 8 * (h.hbm_pages + h.host_pages)) return OR_ERR_INVALID_ARG;
  if (h.world_size != p->c.world_size || h.rank >= p->c.world_size || h.rank == p->c.rank) return OR_ERR_INVALID_ARG;
  if (h.page_bytes != p->c.page_bytes || h.gva_hbm_start != p->c.gva_hbm_start || h.gva_host_start != p->c.gva_host_start ||
      h.max_size != p->c.max_size)
    return OR_ERR_INVALID_ARG;
  or_peer* pr = &p->peers[h.rank];
  if (pr->present) return OR_ERR_SLOT_IN_USE;
  if ((h.hbm_pages && !peer_hbm) || (h.host_pages && !peer_host) || (h.text_pages && !peer_text)) return OR_ERR_INVALID_ARG;
  pr->hbm_pages = h.hbm_pages; pr->host_pages = h.host_pages; pr->text_pages = h.text_pages;
  pr->bind_hbm = (uint64_t*)malloc(8 * (h.hbm_pages + 1));
  pr->bind_host = (uint64_t*)malloc(8 * (h.host_pages + 1));
  memcpy(pr->bind_hbm, (const uint8_t*)buf + sizeof(h), 8 * h.hbm_pages);
  memcpy(pr->bind_host, (const uint8_t*)buf + sizeof(h) + 8 * h.hbm_pages, 8 * h.host_pages);
  pr->hbm_mem = (uint8_t*)peer_hbm; pr->host_mem = (uint8_t*)peer_host; pr->text_mem = (uint8_t*)peer_text;
  pr->present = 1;
  return OR_OK;
}

/* blob: header {magic, n, src_rank}, then per sample: seq_len, n_spans, n_text_pages, its spans (pos, tokens,
 * n_pages, page GVAs...), its text-page GVAs -- all as u64 words */
int32_t oracle_pool_export_samples(oracle_pool* p, const uint32_t* slot, uint32_t n, void* buf, uint64_t cap,
                                   uint64_t* bytes) {
  if (!p || (n && !slot)) return OR_ERR_INVALID_ARG;
  uint64_t words = 3;
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= p->c.max_samples) return OR_ERR_INVALID_ARG;
    const or_sample* s = &p->samples[slot[i]];
    if (s->state == SLOT_FREE) return OR_ERR_UNKNOWN_SAMPLE;
    for (uint32_t j = 0; j < i; ++j)
      if (slot[j] == slot[i]) return OR_ERR_INVALID_ARG;
    if (s->state != SLOT_READY) return OR_ERR_NOT_READY;
    words += 3 + s->n_text_pages;
    for (uint32_t j = 0; j < s->n_spans; ++j) words += 6 + s->spans[j].n_pages; /* pos, tokens, pages, grid T H W */
  }
  if (bytes) *bytes = 8 * words;
  if (!buf) return OR_OK;
  if (cap < 8 * words) return OR_ERR_CAPACITY;
  uint64_t* w = (uint64_t*)buf;
  *w++ = OR_SMP_MAGIC; *w++ = n; *w++ = p->c.rank;
  for (uint32_t i = 0; i < n; ++i) {
    const or_sample* s = &p->samples[slot[i]];
    *w++ = s->seq_len; *w++ = s->n_spans; *w++ = s->n_text_pages;
    for (uint32_t j = 0; j < s->n_spans; ++j) {
      *w++ = s->spans[j].pos_start; *w++ = s->spans[j].n_tokens; *w++ = s->spans[j].n_pages;
      *w++ = s->spans[j].grid[0]; *w++ = s->spans[j].grid[1]; *w++ = s->spans[j].grid[2];
      for (uint32_t o = 0; o < s->spans[j].n_pages; ++o) *w++ = s->spans[j].pages[o];
    }
    for (uint32_t k = 0; k < s->n_text_pages; ++k) *w++ = s->text_pages[k];
  }
  return OR_OK;
}

int32_t oracle_pool_import_samples(oracle_pool* p, const uint32_t* local_slot, uint32_t n, const void* buf,
                                   uint64_t bytes) {
  if (!p || !buf || bytes < 24 || (n && !local_slot)) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  const uint64_t* w = (const uint64_t*)buf;
  const uint64_t* end = w + bytes / 8;
  if (w[0] != OR_SMP_MAGIC || w[1] != n) return OR_ERR_INVALID_ARG;
  if (w[2] >= p->c.world_size || !p->peers[w[2]].present) return OR_ERR_INVALID_ARG; /* mapping first */
  if (n == 0) return OR_OK;
  /* checks, in argument order */
  const uint64_t* r = w + 3;
  for (uint32_t i = 0; i < n; ++i) {
    if (local_slot[i] >= p->c.max_samples) return OR_ERR_INVALID_ARG;
    if (p->samples[local_slot[i]].state != SLOT_FREE) return OR_ERR_SLOT_IN_USE;
    for (uint32_t j = 0; j < i; ++j)
      if (local_slot[j] == local_slot[i]) return OR_ERR_SLOT_IN_USE;
    if (r + 3 > end) return OR_ERR_INVALID_ARG;
    uint64_t seq_len = r[0], n_spans = r[1], ntp = r[2];
    r += 3;
    if (seq_len == 0 || ntp != (seq_len + TEXT_PAGE_IDS - 1) / TEXT_PAGE_IDS) return OR_ERR_INVALID_ARG;
    if (seq_len > p->c.max_seq_len || n_spans > p->c.max_spans_per_sample) return OR_ERR_CAPACITY;
    for (uint64_t j = 0; j < n_spans; ++j) {
      if (r + 6 > end) return OR_ERR_INVALID_ARG;
      uint64_t np = r[2];
      if (np > (uint64_t)((p->c.max_pages_per_span + 63) / 64) * 64) return OR_ERR_CAPACITY;
      /* the span's token grid travels with it: none (all zero), or extents whose product is the token count */
      if (r[3] | r[4] | r[5]) {
        if (!r[3] || !r[4] || !r[5] || r[3] > r[1] || r[4] > r[1] || r[5] > r[1]) return OR_ERR_INVALID_ARG;
        if (r[3] * r[4] > r[1] || r[3] * r[4] * r[5] != r[1]) return OR_ERR_INVALID_ARG;
      }
      r += 6 + np;
    }
    r += ntp;
    if (r > end) return OR_ERR_INVALID_ARG;
  }
  if (r != end) return OR_ERR_INVALID_ARG;
  r = w + 3;
  for (uint32_t i = 0; i < n; ++i) {
    or_sample* s = &p->samples[local_slot[i]];
    s->state = SLOT_READY; s->remote = 1;
    ready_push(p, local_slot[i]);
    s->seq_len = (uint32_t)r[0]; s->n_spans = (uint32_t)r[1]; s->n_text_pages = (uint32_t)r[2];
    s->spans_written = s->n_spans;
    r += 3;
    s->spans = (or_span*)calloc(s->n_spans + 1, sizeof(or_span));
    for (uint32_t j = 0; j < s->n_spans; ++j) {
      s->spans[j].pos_start = (uint32_t)r[0]; s->spans[j].n_tokens = (uint32_t)r[1]; s->spans[j].n_pages = (uint32_t)r[2];
      s->spans[j].grid[0] = (uint32_t)r[3]; s->spans[j].grid[1] = (uint32_t)r[4]; s->spans[j].grid[2] = (uint32_t)r[5];
      r += 6;
      s->spans[j].pages = (uint64_t*)malloc(8 * (s->spans[j].n_pages + 1));
      for (uint32_t o = 0; o < s->spans[j].n_pages; ++o) s->spans[j].pages[o] = *r++;
    }
    s->text_pages = (uint64_t*)malloc(8 * (s->n_text_pages + 1));
    for (uint32_t k = 0; k < s->n_text_pages; ++k) s->text_pages[k] = *r++;
  }
  return OR_OK;
}

static int ready_live(const oracle_pool* p, uint64_t i) {
  const or_sample* s = &p->samples[p->rq_slot[i]];
  return s->state == SLOT_READY && s->generation == p->rq_gen[i];
}

int32_t oracle_pool_ready_count(oracle_pool* p, uint32_t* n_samples, uint64_t* n_tokens) {
  if (!p) return OR_ERR_INVALID_ARG;
  uint32_t n = 0; uint64_t tok = 0;
  for (uint64_t i = p->rq_head; i < p->rq_tail; ++i)
    if (ready_live(p, i)) { ++n; tok += p->samples[p->rq_slot[i]].seq_len; }
  if (n_samples) *n_samples = n;
  if (n_tokens) *n_tokens = tok;
  return OR_OK;
}

/* pops up to max_samples ready samples in completion order once min_tokens tokens are ready; entries of samples
 * freed since are skipped */
int32_t oracle_pool_take_ready(oracle_pool* p, uint64_t min_tokens, uint32_t max_samples, uint32_t* slots_out,
                               uint32_t* n_out, uint64_t* tokens_out) {
  if (!p || !n_out || (max_samples && !slots_out)) return OR_ERR_INVALID_ARG;
  *n_out = 0;
  if (tokens_out) *tokens_out = 0;
  uint64_t avail = 0;
  for (uint64_t i = p->rq_head; i < p->rq_tail; ++i)
    if (ready_live(p, i)) avail += p->samples[p->rq_slot[i]].seq_len;
  if (avail < min_tokens || avail == 0) return OR_ERR_NOT_READY;
  uint32_t n = 0; uint64_t tok = 0;
  while (p->rq_head < p->rq_tail && n < max_samples) {
    uint64_t i = p->rq_head++;
    if (!ready_live(p, i)) continue;
    slots_out[n++] = p->rq_slot[i];
    tok += p->samples[p->rq_slot[i]].seq_len;
  }
  *n_out = n;
  if (tokens_out) *tokens_out = tok;
  return OR_OK;
}

/* ---- accessors for the harness ---- */
int32_t oracle_pool_status(oracle_pool* p, int32_t* code, uint64_t* detail) {
  if (!p) return OR_ERR_INVALID_ARG;
  if (p->status_key == UINT64_MAX) { if (code) *code = 0; if (detail) *detail = 0; return OR_OK; }
  if (code) *code = -(int32_t)((p->status_key >> 32) & 0xFF);
  if (detail) *detail = p->status_key & 0xFFFFFFFFull;
  p->status_key = UINT64_MAX;
  return OR_OK;
}

int32_t oracle_pool_debug_span_pages(oracle_pool* p, uint32_t slot, uint32_t span, uint64_t* gva_out,
                                     uint32_t cap, uint32_t* n) {
  if (!p || slot >= p->c.max_samples) return OR_ERR_INVALID_ARG;
  or_sample* s = &p->samples[slot];
  if (s->state == SLOT_FREE) return OR_ERR_UNKNOWN_SAMPLE;
  if (span >= s->n_spans) return OR_ERR_INVALID_ARG;
  if (n) *n = s->spans[span].n_pages;
  for (uint32_t o = 0; o < s->spans[span].n_pages && o < cap; ++o) gva_out[o] = s->spans[span].pages[o];
  return OR_OK;
}

int32_t oracle_pool_free_pages(oracle_pool* p, uint64_t* n_free, uint64_t* n_text_free) {
  if (!p) return OR_ERR_INVALID_ARG;
  if (n_free) *n_free = p->ring_count;
  if (n_text_free) *n_text_free = p->tring_count;
  return OR_OK;
}

/* the ring's current content, head first */
int32_t oracle_pool_debug_ring(oracle_pool* p, uint32_t* out, uint64_t cap, uint64_t* n) {
  if (!p) return OR_ERR_INVALID_ARG;
  if (n) *n = p->ring_count;
  for (uint64_t i = 0; i < p->ring_count && i < cap; ++i) out[i] = p->ring[(p->ring_head + i) % p->P];
  return OR_OK;
}

/* raw byte of a backing tier, for read-back checks: kind 0 HBM, 1 DRAM */
const uint8_t* oracle_pool_backing(oracle_pool* p, uint32_t kind) {
  return kind == 0 ? p->hbm_mem : kind == 1 ? p->host_mem : p->text_mem;
}

int32_t oracle_plan_summary(const oracle_plan* pl, uint32_t* n_mb, uint64_t* total_tokens, uint32_t* max_mb_tokens) {
  if (!pl) return OR_ERR_INVALID_ARG;
  uint64_t tot = 0; uint32_t mx = 0;
  for (uint32_t j = 0; j < pl->n_mb; ++j) { tot += pl->mb_tokens[j]; if (pl->mb_tokens[j] > mx) mx = pl->mb_tokens[j]; }
  if (n_mb) *n_mb = pl->n_mb;
  if (total_tokens) *total_tokens = tot;
  if (max_mb_tokens) *max_mb_tokens = mx;
  return OR_OK;
}

/* copies every plan array out; any pointer may be NULL */
int32_t oracle_plan_arrays(const oracle_plan* pl, uint32_t* mb_sample_off, uint32_t* mb_samples,
                           uint32_t* mb_tokens, uint32_t* mb_lmax, uint32_t* mb_residual,
                           uint64_t* mb_cost, uint32_t* mb_bucket, uint32_t* mb_rank,
                           uint32_t* rank_mb_off, uint32_t* rank_mbs, uint64_t* sample_cost,
                           uint32_t* sample_mb) {
  if (!pl) return OR_ERR_INVALID_ARG;
  const uint32_t n = pl->n, m = pl->n_mb, N = pl->c.n_ranks_N;
#define CP(dst, src, cnt) if (dst) memcpy(dst, src, (size_t)(cnt) * sizeof(*(src)))
  CP(mb_sample_off, pl->mb_sample_off, m + 1); CP(mb_samples, pl->mb_samples, n);
  CP(mb_tokens, pl->mb_tokens, m); CP(mb_lmax, pl->mb_lmax, m); CP(mb_residual, pl->mb_residual, m);
  CP(mb_cost, pl->mb_cost, m); CP(mb_bucket, pl->mb_bucket, m); CP(mb_rank, pl->mb_rank, m);
  CP(rank_mb_off, pl->rank_mb_off, N + 1); CP(rank_mbs, pl->rank_mbs, m);
  CP(sample_cost, pl->sample_cost, n); CP(sample_mb, pl->sample_mb, n);
  return OR_OK;
}

/* ------------------------------------------------------------------------
 * Backbone-side outputs next to assembly.  The paper stops at "the backbone
 * consumes microbatches"; nothing below has a passage of its own.  What the
 * paper does fix: image and text subsequences are interleaved (Sec. 4.1),
 * a microbatch holds at most L tokens (Sec. 3.4), and the encoders are frozen
 * (Sec. 4.3), so the only gradient that flows back through the assembled
 * input is the embedding table's.  Each function states its own definition;
 * the pins are hand-worked examples and reductions to the packed assembly
 * and to library routines.
 * ---------------------------------------------------------------------- */

/* Token grid of a span: (T, H, W) with T*H*W = n_tokens, row-major (t, h, w).
 * All-or-nothing: the first bad item stops the call and nothing is stored.  Items are stored in order, so of
 * several items naming the same span the last one stays. */
int32_t oracle_pool_set_span_grids(oracle_pool* p, uint32_t n, const uint32_t* slot, const uint32_t* span_idx,
                                   const uint32_t* grid_thw) {
  if (!p) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (n && (!slot || !span_idx || !grid_thw)) return OR_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= p->c.max_samples) return OR_ERR_INVALID_ARG;
    or_sample* s = &p->samples[slot[i]];
    if (s->state == SLOT_FREE) return OR_ERR_UNKNOWN_SAMPLE;
    if (span_idx[i] >= s->n_spans) return OR_ERR_INVALID_ARG;
    const uint32_t* g = grid_thw + 3ull * i;
    if (g[0] == 0 || g[1] == 0 || g[2] == 0) return OR_ERR_INVALID_ARG;
    if ((uint64_t)g[0] * g[1] * g[2] != s->spans[span_idx[i]].n_tokens) return OR_ERR_INVALID_ARG;
  }
  for (uint32_t i = 0; i < n; ++i)
    memcpy(p->samples[slot[i]].spans[span_idx[i]].grid, grid_thw + 3ull * i, 12);
  return OR_OK;
}

/* Three-component position of every token of one sample (the multimodal rotary scheme of current
 * vision-language backbones): a counter st starts at 0; a text token gets (st, st, st) and st += 1; a span
 * with grid (T, H, W) starting at counter st gives its token (t, h, w) the position (st + t, st + h, st + w)
 * and then st += max(T, H, W); a span without a grid counts as text. */
static void sample_positions3(const or_sample* s, int32_t* out /* [seq_len][3] */) {
  int64_t st = 0;
  uint32_t pos = 0;
  while (pos < s->seq_len) {
    const or_span* sp = NULL;
    for (uint32_t i = 0; i < s->n_spans; ++i)
      if (pos >= s->spans[i].pos_start && pos < s->spans[i].pos_start + s->spans[i].n_tokens) sp = &s->spans[i];
    if (sp && sp->grid[0] && pos == sp->pos_start) {
      const uint32_t T = sp->grid[0], H = sp->grid[1], W = sp->grid[2];
      for (uint32_t t = 0; t < T; ++t)
        for (uint32_t h = 0; h < H; ++h)
          for (uint32_t w = 0; w < W; ++w, ++pos) {
            out[3ull * pos + 0] = (int32_t)(st + t); out[3ull * pos + 1] = (int32_t)(st + h); out[3ull * pos + 2] = (int32_t)(st + w);
          }
      uint32_t m = T; if (H > m) m = H; if (W > m) m = W;
      st += m;
    } else {
      out[3ull * pos + 0] = out[3ull * pos + 1] = out[3ull * pos + 2] = (int32_t)st;
      ++st; ++pos;
    }
  }
}

#define OR_IGNORE_LABEL (-100)

/* Padded assembly: every microbatch of [mb_begin, mb_end) occupies exactly L rows.
 *   out_embeds [(mb_end-mb_begin)*L][H] bf16: the packed rows of the microbatch, then zero rows;
 *   out_cu_seqlens: per microbatch n_j + 2 entries: 0, the sample ends, then L (the padding as one last sequence,
 *     of length 0 when the microbatch is full);
 *   out_pos3 [3][rows]: component-major three-component positions (0 on padding rows);
 *   out_ids [rows]: the token id of the position (the id stored at a placeholder position included), pad_id on padding;
 *   out_labels [rows]: next-token target: the id at the following position of the same sample when that
 *     position is a text position (not inside a span), else -100; -100 on the last position and on padding;
 *   out_mask [rows] bytes: 1 where the label is not -100.
 * Errors as oracle_pool_gather_packed; detail of an asynchronous error = padded row index. */
int32_t oracle_pool_gather_padded(oracle_pool* p, const oracle_plan* pl, uint32_t mb_begin, uint32_t mb_end,
                                  const void* embed_table, uint32_t vocab, int32_t pad_id, void* out_embeds,
                                  int32_t* out_cu_seqlens, int32_t* out_pos3, int32_t* out_ids, int32_t* out_labels,
                                  uint8_t* out_mask) {
  if (!p || !pl) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (mb_begin > mb_end || mb_end > pl->n_mb) return OR_ERR_INVALID_ARG;
  for (uint32_t t = 0; t < pl->n; ++t) {
    or_sample* s = &p->samples[pl->slots[t]];
    if (s->state != SLOT_READY || s->generation != pl->slot_generation[t]) return OR_ERR_NOT_READY;
  }
  if (mb_begin == mb_end) return OR_OK;
  if (!embed_table || !out_embeds || !out_cu_seqlens || !out_pos3 || !out_ids || !out_labels || !out_mask)
    return OR_ERR_INVALID_ARG;
  const uint64_t PS = p->c.page_bytes, row_bytes = 2ull * p->c.hidden, L = pl->c.budget_L;
  const uint64_t rows = (uint64_t)(mb_end - mb_begin) * L;
  uint8_t* out = (uint8_t*)out_embeds;
  uint64_t cu_w = 0;
  for (uint32_t j = mb_begin; j < mb_end; ++j) {
    uint64_t row = (uint64_t)(j - mb_begin) * L;
    const uint64_t row_end = row + L;
    int32_t cu = 0;
    out_cu_seqlens[cu_w++] = 0;
    for (uint32_t qi = pl->mb_sample_off[j]; qi < pl->mb_sample_off[j + 1]; ++qi) {
      or_sample* s = &p->samples[pl->mb_samples[qi]];
      int32_t* p3 = (int32_t*)calloc(3ull * s->seq_len + 3, sizeof(int32_t));
      int32_t* ids = (int32_t*)calloc((size_t)s->seq_len + 1, sizeof(int32_t));
      uint8_t* vis = (uint8_t*)calloc((size_t)s->seq_len + 1, 1);
      sample_positions3(s, p3);
      for (uint32_t pos = 0; pos < s->seq_len; ++pos) {
        memcpy(&ids[pos], resolve(p, s->text_pages[pos / TEXT_PAGE_IDS] + (uint64_t)(pos % TEXT_PAGE_IDS) * 4), 4);
        for (uint32_t i = 0; i < s->n_spans; ++i)
          if (pos >= s->spans[i].pos_start && pos < s->spans[i].pos_start + s->spans[i].n_tokens) vis[pos] = 1;
      }
      for (uint32_t pos = 0; pos < s->seq_len; ++pos, ++row) {
        for (int c = 0; c < 3; ++c) out_pos3[(uint64_t)c * rows + row] = p3[3ull * pos + c];
        out_ids[row] = ids[pos];
        const int has_label = pos + 1 < s->seq_len && !vis[pos + 1];
        out_labels[row] = has_label ? ids[pos + 1] : OR_IGNORE_LABEL;
        out_mask[row] = (uint8_t)has_label;
        uint8_t* dst = out + row * row_bytes;
        if (vis[pos]) {
          const or_span* sp = NULL;
          for (uint32_t i = 0; i < s->n_spans; ++i)
            if (pos >= s->spans[i].pos_start && pos < s->spans[i].pos_start + s->spans[i].n_tokens) sp = &s->spans[i];
          uint64_t b = (uint64_t)(pos - sp->pos_start) * row_bytes, done = 0;
          while (done < row_bytes) {
            uint64_t off = (b + done) % PS;
            uint64_t run = PS - off < row_bytes - done ? PS - off : row_bytes - done;
            uint8_t* src = resolve(p, sp->pages[(b + done) / PS] + off);
            if (!src) { note_async_error(p, OR_ERR_BAD_GVA, (uint32_t)row); break; }
            memcpy(dst + done, src, run);
            done += run;
          }
        } else if (ids[pos] < 0 || (uint32_t)ids[pos] >= vocab) {
          note_async_error(p, OR_ERR_BAD_TOKEN_ID, (uint32_t)row); /* row left untouched */
        } else {
          memcpy(dst, (const uint8_t*)embed_table + (uint64_t)ids[pos] * row_bytes, row_bytes);
        }
      }
      free(p3); free(ids); free(vis);
      cu += (int32_t)s->seq_len;
      out_cu_seqlens[cu_w++] = cu;
    }
    out_cu_seqlens[cu_w++] = (int32_t)L;
    for (; row < row_end; ++row) { /* padding */
      memset(out + row * row_bytes, 0, row_bytes);
      for (int c = 0; c < 3; ++c) out_pos3[(uint64_t)c * rows + row] = 0;
      out_ids[row] = pad_id; out_labels[row] = OR_IGNORE_LABEL; out_mask[row] = 0;
    }
  }
  return OR_OK;
}

static float bf16_bits_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* Gradient of the embedding table through the assembled input.  grad_out holds one bf16 row per output row of
 * the range, in the packed layout (padded = 0) or the L-rows-per-microbatch layout (padded != 0).  For the rows in
 * ascending order: a row at a text position with id v adds its values, widened exactly to fp32, to row v of
 * grad_table with one fp32 addition per element; rows at span positions (frozen encoders) and padding rows add
 * nothing.  The order of the additions is part of the definition: fp32 addition is not associative. */
int32_t oracle_pool_embed_grad(oracle_pool* p, const oracle_plan* pl, uint32_t mb_begin, uint32_t mb_end,
                               int padded, const void* grad_out, float* grad_table, uint32_t vocab) {
  if (!p || !pl) return OR_ERR_INVALID_ARG;
  p->call_seq++;
  if (mb_begin > mb_end || mb_end > pl->n_mb) return OR_ERR_INVALID_ARG;
  for (uint32_t t = 0; t < pl->n; ++t) {
    or_sample* s = &p->samples[pl->slots[t]];
    if (s->state != SLOT_READY || s->generation != pl->slot_generation[t]) return OR_ERR_NOT_READY;
  }
  if (mb_begin == mb_end) return OR_OK;
  if (!grad_out || !grad_table) return OR_ERR_INVALID_ARG;
  const uint64_t H = p->c.hidden, L = pl->c.budget_L;
  const uint16_t* g = (const uint16_t*)grad_out;
  uint64_t row = 0;
  for (uint32_t j = mb_begin; j < mb_end; ++j) {
    if (padded) row = (uint64_t)(j - mb_begin) * L;
    for (uint32_t qi = pl->mb_sample_off[j]; qi < pl->mb_sample_off[j + 1]; ++qi) {
      or_sample* s = &p->samples[pl->mb_samples[qi]];
      for (uint32_t pos = 0; pos < s->seq_len; ++pos, ++row) {
        int vis = 0;
        for (uint32_t i = 0; i < s->n_spans; ++i)
          if (pos >= s->spans[i].pos_start && pos < s->spans[i].pos_start + s->spans[i].n_tokens) vis = 1;
        if (vis) continue;
        int32_t id;
        memcpy(&id, resolve(p, s->text_pages[pos / TEXT_PAGE_IDS] + (uint64_t)(pos % TEXT_PAGE_IDS) * 4), 4);
        if (id < 0 || (uint32_t)id >= vocab) { note_async_error(p, OR_ERR_BAD_TOKEN_ID, (uint32_t)row); continue; }
        float* dst = grad_table + (uint64_t)id * H;
        const uint16_t* src = g + row * H;
        for (uint64_t c = 0; c < H; ++c) {
          volatile float sum = dst[c] + bf16_bits_to_f32(src[c]); /* one rounded fp32 addition */
          dst[c] = sum;
        }
      }
    }
  }
  return OR_OK;
}
