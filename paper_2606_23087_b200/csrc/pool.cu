// Pool life cycle, registration, page allocation, producer scatter and free (sm_100a).
//
// Kernels in this file
//   k_page_table_init  PTEs from the vpn->frame binding (Sec. 3.2: page tables map GVA -> physical)
//   k_register_scan    per-sample text-page counts -> exclusive scan, sample + span tables, text-page pops and records
//   k_register_ids     token ids into text pages, placeholder-run validation
//   k_alloc_scan       pages/list blocks/chunks per span -> exclusive scans, ring pops
//   k_alloc_fill       span page lists (two-level) from consecutive ring entries; chunk records for k_scatter
//   k_scatter          the producer byte copy into pages, optional fused fp32->bf16 RNE cast
//   k_scatter_host_bulk  bf16 sources into host-tier pages by bulk-async copies
//   k_free_scan/_fill  pages, list blocks and text pages back to the ring tails
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <unordered_set>

#include "bulk_copy.cuh"
#include "flowpool_internal.cuh"

namespace ft {

// one caller thread per pool, so a per-thread string is per pool as far as any caller can tell
static thread_local char g_last_error[512] = "";

static std::mutex g_pools_mu;
static std::unordered_set<ft_pool*> g_pools;
void pool_registry_add(ft_pool* p) { std::lock_guard<std::mutex> l(g_pools_mu); g_pools.insert(p); }
void pool_registry_remove(ft_pool* p) { std::lock_guard<std::mutex> l(g_pools_mu); g_pools.erase(p); }
bool pool_registry_has(ft_pool* p) { std::lock_guard<std::mutex> l(g_pools_mu); return g_pools.count(p) != 0; }

int32_t cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_last_error, sizeof(g_last_error), "%s: %s", what, cudaGetErrorString(e));
  cudaGetLastError();
  return FT_ERR_CUDA;
}

// Counter-based hash of the seeded shuffles: the published SplitMix64 finaliser,
// hash(seed, i) = mix(seed ^ mix(i)); Fisher-Yates runs i = n-1..1 with j = hash mod (i+1).
static inline uint64_t mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
static void seeded_shuffle(std::vector<uint32_t>& a, uint64_t seed) {
  for (uint64_t i = a.size(); i-- > 1;) {
    uint64_t j = mix64(seed ^ mix64(i)) % (i + 1);
    std::swap(a[i], a[j]);
  }
}

int32_t ctx_acquire(ft_pool* p, int side, size_t blob_bytes, size_t total_bytes, ft_call_ctx** out, bool on_meta, cudaStream_t first_user) {
  ft_call_ctx& c = p->ctx[side][p->ctx_next[side]];
  p->ctx_next[side] = (p->ctx_next[side] + 1) % kCallCtx;
  if (c.busy_up) { FT_CUDA(cudaEventSynchronize(c.ev_up)); c.busy_up = false; }  // the upload that last read `h` is over
  if (c.hcap < blob_bytes) {
    if (c.h) FT_CUDA(cudaFreeHost(c.h));
    size_t cap = 1 << 16;
    while (cap < blob_bytes) cap <<= 1;
    c.h = nullptr; c.hcap = 0;
    FT_CUDA(cudaHostAlloc(&c.h, cap, cudaHostAllocMapped));
    FT_CUDA(cudaHostGetDevicePointer(&c.hd, c.h, 0));
    c.hcap = cap;
  }
  if (c.dcap < total_bytes) {
    // a call larger than any before it on this side: every context of the side grows now (allocating synchronises
    // the device; once for all of them instead of once per context as the ring comes round)
    size_t cap = 1 << 18;
    while (cap < total_bytes) cap <<= 1;
    for (int i = 0; i < kCallCtx; ++i) {
      ft_call_ctx& g = p->ctx[side][i];
      if (g.dcap >= cap) continue;
      if (g.busy_done) { FT_CUDA(cudaEventSynchronize(g.ev_done)); g.busy_done = false; }  // nobody reads the old scratch
      if (g.d) FT_CUDA(cudaFree(g.d));
      g.d = nullptr; g.dcap = 0;
      FT_CUDA(cudaMalloc(&g.d, cap));
      g.dcap = cap;
    }
  }
  if (c.busy_done) { FT_CUDA(cudaStreamWaitEvent(on_meta ? p->meta : first_user, c.ev_done, 0)); c.busy_done = false; }
  *out = &c;
  return FT_OK;
}

// The library's own small transfers (a call's descriptors up, a plan's summary down) are made by a kernel that reads or
// writes mapped pinned memory, not by cudaMemcpyAsync: the copy engines serve their queues in order, so a descriptor
// upload behind an application's bulk host-to-device copy (or a plan's summary behind a bulk copy-out) would wait for
// all of it, and every call of the pool with it.
__global__ void k_copy_words(uint32_t* __restrict__ dst, const uint32_t* __restrict__ src, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) dst[i] = src[i];
}
int32_t copy_words(void* dst, const void* src, size_t n_words, cudaStream_t st) {
  if (n_words == 0) return FT_OK;
  const unsigned grid = (unsigned)std::min<size_t>((n_words + 255) / 256, 64);
  k_copy_words<<<grid, 256, 0, st>>>(static_cast<uint32_t*>(dst), static_cast<const uint32_t*>(src), n_words);
  FT_CUDA(cudaGetLastError());
  return FT_OK;
}

int32_t ctx_upload(ft_pool* p, ft_call_ctx* c, size_t bytes) {
  p->meta_seq++;
  if (bytes) {
    const int32_t rc = copy_words(c->d, c->hd, (bytes + 3) / 4, p->meta);
    if (rc != FT_OK) return rc;
    p->gpu_launches++;
    FT_CUDA(cudaEventRecord(c->ev_up, p->meta));
    c->busy_up = true;
  }
  return FT_OK;
}

int32_t ctx_release(ft_pool* p, ft_call_ctx* c, cudaStream_t last) {
  (void)p;
  FT_CUDA(cudaEventRecord(c->ev_done, last));
  c->busy_done = true;
  return FT_OK;
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
size_t align_up_sz(size_t x, size_t a) { return align_up(x, a); }

// ------------------------------------------------------------------------------------------
// K1: page tables
// ------------------------------------------------------------------------------------------
__global__ void k_page_table_init(uint64_t* pte, const uint32_t* bind, uint64_t n, uint64_t base, uint64_t frame_bytes,
                                  uint64_t flags) {
  uint64_t v = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v < n) pte[v] = (base + (bind ? (uint64_t)bind[v] : v) * frame_bytes) | flags;
}

__global__ void k_iota(uint32_t* a, uint64_t n) {
  uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) a[i] = (uint32_t)i;
}

// ------------------------------------------------------------------------------------------
// K2: registration
// ------------------------------------------------------------------------------------------
struct RegisterCall {
  uint32_t n;
  const uint32_t *slot, *seq_len, *n_spans, *span_begin;  // [n], [n], [n], [n+1]
  const uint64_t* ids_off;                                // [n+1]
  const uint32_t *span_pos, *span_tok;                    // concatenated
  const int32_t* ids;                                     // device, concatenated
  uint32_t* tp_off;                                       // [n+1] out: exclusive scan of text pages
  uint32_t* head;                                         // [1]   out: text ring head before the pops
  uint32_t* pg_sample;                                    // [text pages of the call] out: call-local sample of each page
  uint64_t* pg_dst;                                       // [text pages of the call] out: frame address of each page
  uint64_t call_seq;
};

__global__ void __launch_bounds__(1024) k_register_scan(PoolView v, RegisterCall c) {
  uint64_t carry = 0;
  for (uint32_t base = 0; base < c.n; base += blockDim.x) {
    uint32_t i = base + threadIdx.x;
    uint64_t ntp = 0;
    if (i < c.n) {
      ntp = (c.seq_len[i] + kTextPageIds - 1) / kTextPageIds;
      const uint32_t slot = c.slot[i];
      v.s_seq_len[slot] = c.seq_len[i];
      v.s_n_spans[slot] = c.n_spans[i];
      v.s_flags[slot] = 0;
      for (uint32_t j = 0; j < c.n_spans[i]; ++j) {
        const uint32_t sid = slot * v.spans_per_sample + j;
        v.sp_pos[sid] = c.span_pos[c.span_begin[i] + j];
        v.sp_tokens[sid] = c.span_tok[c.span_begin[i] + j];
        v.sp_npages[sid] = 0;
        v.sp_grid[sid] = make_uint4(0, 0, 0, 0);
      }
    }
    uint64_t total, ex = block_exclusive_scan(ntp, &total);
    if (i < c.n) c.tp_off[i] = (uint32_t)(carry + ex);
    carry += total;
  }
  __shared__ uint32_t sh_head;
  if (threadIdx.x == 0) {
    c.tp_off[c.n] = (uint32_t)carry;
    RingState s = *v.tring_state;
    c.head[0] = s.head;
    sh_head = s.head;
    s.head = (uint32_t)((s.head + carry) % v.tring_cap);
    s.count -= (uint32_t)carry;
    *v.tring_state = s;
  }
  __syncthreads();
  // every text page of the call: which sample it serves and where it lives, so that the copy of the ids (on the
  // caller's stream, between its data kernels) starts from one small record instead of a search and three lookups
  for (uint32_t b = threadIdx.x; b < (uint32_t)carry; b += blockDim.x) {
    uint32_t lo = 0, hi = c.n;  // largest i with tp_off[i] <= b
    while (hi - lo > 1) {
      uint32_t mid = (lo + hi) >> 1;
      if (c.tp_off[mid] <= b) lo = mid; else hi = mid;
    }
    const uint32_t tp = v.tring[(sh_head + b) % v.tring_cap];
    const uint64_t tp_gva = v.text_gva_base + (uint64_t)tp * FT_TEXT_PAGE_BYTES;
    v.s_text_pages[(uint64_t)c.slot[lo] * v.text_pages_per_sample + (b - c.tp_off[lo])] = tp_gva;
    uint64_t off;
    c.pg_sample[b] = lo;
    c.pg_dst[b] = translate(v, tp_gva, &off) & ~kPteFlagMask;
  }
}

// one block per (sample, text page): stores up to 1024 ids, validates the runs
__global__ void __launch_bounds__(256) k_register_ids(PoolView v, RegisterCall c) {
  const uint32_t b = blockIdx.x;
  const uint32_t i = c.pg_sample[b], k = b - c.tp_off[i], slot = c.slot[i];
  int32_t* dst = reinterpret_cast<int32_t*>(c.pg_dst[b]);
  const uint32_t len = c.seq_len[i], p0 = k * kTextPageIds;
  const uint32_t cnt = min(kTextPageIds, len - p0);
  const uint32_t sb = c.span_begin[i], ns = c.n_spans[i];
  bool bad = false;
  for (uint32_t t = threadIdx.x; t < cnt; t += blockDim.x) {
    const uint32_t p = p0 + t;
    const int32_t id = c.ids[c.ids_off[i] + p];
    dst[t] = id;
    // is p inside a placeholder run?  last span with pos <= p
    uint32_t lo = 0, hi = ns;
    while (lo < hi) {
      uint32_t mid = (lo + hi) >> 1;
      if (c.span_pos[sb + mid] <= p) lo = mid + 1; else hi = mid;
    }
    const bool in_run = lo > 0 && p < c.span_pos[sb + lo - 1] + c.span_tok[sb + lo - 1];
    bad |= (id == v.placeholder_id) != in_run;
  }
  if (bad) note_error(v, c.call_seq, FT_ERR_PLACEHOLDER_MISMATCH, slot);
}

// ------------------------------------------------------------------------------------------
// K3: page allocation
// ------------------------------------------------------------------------------------------
// A scatter work unit resolved ahead of the copy (chunks never straddle a page when the page is at least a chunk).
struct ChunkDesc {
  uint64_t src;       // the span's source
  uint64_t dst;       // frame address + offset of the chunk inside its page | page-table flags (low 4 bits)
  uint32_t ch_local;  // index of the chunk inside the span's image
  uint32_t len;       // bytes of the image in this chunk
};

struct WriteCall {
  uint32_t n;
  const uint64_t* src;       // [n] device pointers
  const uint32_t* span_id;   // [n]
  const uint32_t* n_tokens;  // [n]
  uint32_t* page_off;        // [n+1] out
  uint32_t* blk_off;         // [n+1] out
  uint64_t* chunk_off;       // [n+1] out
  uint32_t* chunk_span;      // [total chunks] out: call-local span index of each chunk; NULL = search chunk_off
  struct ChunkDesc* chunk_desc;  // [total chunks] out: where each chunk comes from and goes to (pages >= chunk), or NULL
  uint32_t* heads;           // [2]   out: page ring head, block ring head before the pops
  uint32_t chunk_shift;      // scatter work unit = 2^chunk_shift bytes of a span's image
};

__global__ void __launch_bounds__(1024) k_alloc_scan(PoolView v, WriteCall c) {
  uint64_t cp = 0, cb = 0, cc = 0;
  for (uint32_t base = 0; base < c.n; base += blockDim.x) {
    uint32_t q = base + threadIdx.x;
    uint64_t k = 0, nb = 0, nc = 0;
    if (q < c.n) {
      const uint64_t bytes = (uint64_t)c.n_tokens[q] * v.row_bytes;
      k = (bytes + v.page_bytes - 1) >> v.page_shift;
      nb = (k + kListBlock - 1) / kListBlock;
      nc = (bytes + (1ull << c.chunk_shift) - 1) >> c.chunk_shift;
      v.sp_npages[c.span_id[q]] = (uint32_t)k;
    }
    uint64_t tp, tb, tc;
    uint64_t ep = block_exclusive_scan(k, &tp);
    uint64_t eb = block_exclusive_scan(nb, &tb);
    uint64_t ec = block_exclusive_scan(nc, &tc);
    if (q < c.n) { c.page_off[q] = (uint32_t)(cp + ep); c.blk_off[q] = (uint32_t)(cb + eb); c.chunk_off[q] = cc + ec; }
    cp += tp; cb += tb; cc += tc;
  }
  if (threadIdx.x == 0) {
    c.page_off[c.n] = (uint32_t)cp; c.blk_off[c.n] = (uint32_t)cb; c.chunk_off[c.n] = cc;
    RingState s = *v.ring_state;
    c.heads[0] = s.head;
    s.head = (uint32_t)((s.head + cp) % v.ring_cap); s.count -= (uint32_t)cp;
    *v.ring_state = s;
    s = *v.bring_state;
    c.heads[1] = s.head;
    s.head = (uint32_t)((s.head + cb) % v.bring_cap); s.count -= (uint32_t)cb;
    *v.bring_state = s;
  }
}

// one thread per allocated page: span q takes ring entries [page_off[q], page_off[q+1]) after the head
__global__ void __launch_bounds__(256) k_alloc_fill(PoolView v, WriteCall c, uint32_t total_pages, uint64_t total_chunks) {
  const uint64_t tc = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c.chunk_span && tc < total_chunks) {  // which span of the call does chunk tc belong to
    uint32_t lo = 0, hi = c.n;
    while (hi - lo > 1) {
      uint32_t mid = (lo + hi) >> 1;
      if (c.chunk_off[mid] <= tc) lo = mid; else hi = mid;
    }
    c.chunk_span[tc] = lo;
    if (c.chunk_desc) {
      const uint32_t ch_local = (uint32_t)(tc - c.chunk_off[lo]);
      const uint64_t B0 = (uint64_t)ch_local << c.chunk_shift, bytes_q = (uint64_t)c.n_tokens[lo] * v.row_bytes;
      const uint32_t g = v.ring[(c.heads[0] + c.page_off[lo] + (uint32_t)(B0 >> v.page_shift)) % v.ring_cap];
      uint64_t off;
      const uint64_t pte = translate(v, page_gva(v, g), &off);
      ChunkDesc d;
      d.src = c.src[lo];
      d.dst = ((pte & ~kPteFlagMask) + (B0 & (v.page_bytes - 1))) | (pte & kPteFlagMask);
      d.ch_local = ch_local;
      d.len = (uint32_t)min((uint64_t)1 << c.chunk_shift, bytes_q - B0);
      c.chunk_desc[tc] = d;
    }
  }
  if (tc >= total_pages) return;
  const uint32_t t = (uint32_t)tc;
  uint32_t lo = 0, hi = c.n;  // largest q with page_off[q] <= t
  while (hi - lo > 1) {
    uint32_t mid = (lo + hi) >> 1;
    if (c.page_off[mid] <= t) lo = mid; else hi = mid;
  }
  const uint32_t q = lo, o = t - c.page_off[q], sid = c.span_id[q];
  const uint32_t g = v.ring[(c.heads[0] + t) % v.ring_cap];
  const uint32_t blk = v.bring[(c.heads[1] + c.blk_off[q] + o / kListBlock) % v.bring_cap];
  if (o % kListBlock == 0) v.sp_blocks[(uint64_t)sid * v.blocks_per_span + o / kListBlock] = blk;
  v.list_blocks[(uint64_t)blk * kListBlock + o % kListBlock] = page_gva(v, g);
}

// ------------------------------------------------------------------------------------------
// K4: producer scatter.  Work unit = one chunk of a span's image.  Where pages are at least a chunk long the chunk
// is one record (source, destination frame + offset, length) that k_alloc_fill prepared; else the CTA finds the
// chunk's span by table or search and each warp resolves its destination frame through the span's page list and
// the page table once per page.  16-byte vectors either way.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t rne_bf16(uint32_t u) {
  // IEEE round-to-nearest-even on the bit pattern; NaN -> sign | 0x7FC0; denormals kept
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return ((u >> 16) & 0x8000u) | 0x7FC0u;
  return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ uint32_t pack2(uint32_t a, uint32_t b) { return rne_bf16(a) | (rne_bf16(b) << 16); }

enum { kTierAll = 0, kTierDeviceOnly = 1, kTierHostOnly = 2 };

// One warp moves up to 2 KiB of a span's image (nv 16-byte vectors, <= 128) from byte offset B of the source image
// (an fp32 source holds two vectors per bf16 vector) to d: four 512-byte lines per lane in flight.
template <bool F32>
__device__ __forceinline__ void copy_batch(const uint8_t* src_q, uint64_t B, uint4* d, uint32_t nv, uint32_t lane) {
  const bool t0 = lane < nv, t1 = lane + 32 < nv, t2 = lane + 64 < nv, t3 = lane + 96 < nv;
  if (!F32) {
    const uint4* s = reinterpret_cast<const uint4*>(src_q + B);
    uint4 a0, a1, a2, a3;
    if (t0) a0 = __ldcs(s + lane);
    if (t1) a1 = __ldcs(s + lane + 32);
    if (t2) a2 = __ldcs(s + lane + 64);
    if (t3) a3 = __ldcs(s + lane + 96);
    if (t0) __stcs(d + lane, a0);
    if (t1) __stcs(d + lane + 32, a1);
    if (t2) __stcs(d + lane + 64, a2);
    if (t3) __stcs(d + lane + 96, a3);
  } else {
    const uint4* s = reinterpret_cast<const uint4*>(src_q + 2 * B);  // two fp32 vectors per bf16 vector
    uint4 a0, a1, a2, a3, e0, e1, e2, e3;
    if (t0) { a0 = __ldcs(s + 2 * lane); e0 = __ldcs(s + 2 * lane + 1); }
    if (t1) { a1 = __ldcs(s + 2 * (lane + 32)); e1 = __ldcs(s + 2 * (lane + 32) + 1); }
    if (t2) { a2 = __ldcs(s + 2 * (lane + 64)); e2 = __ldcs(s + 2 * (lane + 64) + 1); }
    if (t3) { a3 = __ldcs(s + 2 * (lane + 96)); e3 = __ldcs(s + 2 * (lane + 96) + 1); }
    if (t0) __stcs(d + lane, make_uint4(pack2(a0.x, a0.y), pack2(a0.z, a0.w), pack2(e0.x, e0.y), pack2(e0.z, e0.w)));
    if (t1) __stcs(d + lane + 32, make_uint4(pack2(a1.x, a1.y), pack2(a1.z, a1.w), pack2(e1.x, e1.y), pack2(e1.z, e1.w)));
    if (t2) __stcs(d + lane + 64, make_uint4(pack2(a2.x, a2.y), pack2(a2.z, a2.w), pack2(e2.x, e2.y), pack2(e2.z, e2.w)));
    if (t3) __stcs(d + lane + 96, make_uint4(pack2(a3.x, a3.y), pack2(a3.z, a3.w), pack2(e3.x, e3.y), pack2(e3.z, e3.w)));
  }
}

template <int MODE, bool F32, bool DESC>
__global__ void __launch_bounds__(256, F32 ? 4 : 6) k_scatter(PoolView v, WriteCall c, uint64_t total_chunks, uint64_t per_cta,
                                                              ClaimCounter* group_counter) {
  // Work unit = a chunk of 2^chunk_shift bytes of one span's image (the page size does not cap it).  Groups of
  // per_cta consecutive chunks are claimed in order from a device counter (zero at rest: the grid's last CTA puts
  // it back), so at any moment the grid streams one compact window of the call's bytes.  Inside a chunk warp w owns the w-th eighth and walks it in 2 KiB
  // batches (four 512-byte lines per lane in flight); a batch never straddles a page (pages are >= 4 KiB and
  // batches 2 KiB-aligned), and each warp resolves its batch's frame through the span's page list and the
  // page table, once per page.
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint64_t CH = 1ull << c.chunk_shift;
  const uint32_t region = (uint32_t)(CH >> 3);  // bytes per warp and chunk
  // A CTA's first group is its block index; every later one comes from the counter, claimed while the current group
  // is being copied (the answer is needed only when the group is done).
  __shared__ uint64_t next_group[2];
  uint64_t grp = blockIdx.x;
  for (uint32_t it = 0;; ++it) {
    const uint64_t c0 = grp * per_cta;
    if (c0 >= total_chunks) {
      if (threadIdx.x == 0) claim_release(group_counter);
      break;
    }
    unsigned long long nxt = 0;
    if (DESC && threadIdx.x == 0) nxt = gridDim.x + atomicAdd(&group_counter->claim, 1ull);
    const uint64_t c1 = min(total_chunks, c0 + per_cta);
    if (DESC) {
      // resolved chunks: one record, then the bytes
      for (uint64_t ch = c0; ch < c1; ++ch) {
        const ChunkDesc d = c.chunk_desc[ch];
        const bool host = (d.dst & kPteHost) != 0;
        if ((MODE == kTierDeviceOnly && host) || (MODE == kTierHostOnly && !host)) continue;
        const uint64_t B0 = (uint64_t)d.ch_local << c.chunk_shift;
        const uint8_t* src_q = reinterpret_cast<const uint8_t*>(d.src);
        uint8_t* dst0 = reinterpret_cast<uint8_t*>(d.dst & ~kPteFlagMask);
        for (uint32_t b = 0; b < region; b += 2048) {
          const uint32_t Bl = warp * region + b;  // offset inside the chunk
          if (Bl >= d.len) break;
          copy_batch<F32>(src_q, B0 + Bl, reinterpret_cast<uint4*>(dst0 + Bl), (min(2048u, d.len - Bl)) >> 4, lane);
        }
      }
      if (threadIdx.x == 0) next_group[it & 1] = nxt;
      __syncthreads();
      grp = next_group[it & 1];
      continue;
    }
    uint32_t q;
    if (c.chunk_span) {
      q = c.chunk_span[c0];
    } else {
      uint32_t lo = 0, hi = c.n;  // largest q with chunk_off[q] <= c0
      while (hi - lo > 1) {
        uint32_t mid = (lo + hi) >> 1;
        if (c.chunk_off[mid] <= c0) lo = mid; else hi = mid;
      }
      q = lo;
    }
    uint64_t q_end = c.chunk_off[q + 1], q_begin = c.chunk_off[q];
    uint64_t bytes_q = (uint64_t)c.n_tokens[q] * v.row_bytes;
    const uint8_t* src_q = reinterpret_cast<const uint8_t*>(c.src[q]);
    uint32_t sid = c.span_id[q];
    uint32_t cached_o = kNone;
    uint64_t pte = 0;
    for (uint64_t ch = c0; ch < c1; ++ch) {
      while (ch >= q_end) {
        ++q;
        q_begin = q_end; q_end = c.chunk_off[q + 1];
        bytes_q = (uint64_t)c.n_tokens[q] * v.row_bytes;
        src_q = reinterpret_cast<const uint8_t*>(c.src[q]);
        sid = c.span_id[q];
        cached_o = kNone;
      }
      const uint64_t b0 = ((ch - q_begin) << c.chunk_shift) + (uint64_t)warp * region;  // this warp's span offset
      for (uint32_t b = 0; b < region; b += 2048) {
        const uint64_t B = b0 + b;
        if (B >= bytes_q) break;
        const uint32_t o = (uint32_t)(B >> v.page_shift);
        if (o != cached_o) {
          uint64_t off;
          pte = translate(v, span_page_gva(v, sid, o), &off);
          cached_o = o;
        }
        const bool host = (pte & kPteHost) != 0;
        if ((MODE == kTierDeviceOnly && host) || (MODE == kTierHostOnly && !host)) continue;
        uint4* d = reinterpret_cast<uint4*>((pte & ~kPteFlagMask) + (B & (v.page_bytes - 1)));
        copy_batch<F32>(src_q, B, d, (uint32_t)(min((uint64_t)2048, bytes_q - B) >> 4), lane);
      }
    }
    if (threadIdx.x == 0) nxt = gridDim.x + atomicAdd(&group_counter->claim, 1ull);
    if (threadIdx.x == 0) next_group[it & 1] = nxt;
    __syncthreads();
    grp = next_group[it & 1];
  }
}


// launches k_scatter<MODE, F32, records> on a grid of at most `max_ctas` CTAs, never more than fit on the GPU at once
template <int MODE, bool F32>
static void launch_scatter(ft_pool* p, const WriteCall& w, uint64_t total_chunks, uint64_t max_ctas, cudaStream_t s,
                           ClaimCounter* counters) {
  // one claim counter per stream the call launches on: main ([0]) and side ([1])
  ClaimCounter* counter = counters + (s == p->side_stream[0] ? 1 : 0);
  const int per_sm = std::max(1, p->occ_scatter[MODE][F32 ? 1 : 0]);
  // HBM streams best with a bounded amount of loads in flight per SM; more resident warps only deepen the DRAM
  // queues (measured optimum: 4 CTAs/SM, one chunk per claim)
  const int want = p->scatter_ctas_per_sm > 0 ? p->scatter_ctas_per_sm : 4;
  uint64_t grid = std::min<uint64_t>(max_ctas, (uint64_t)p->sm_count * std::min(per_sm, want));
  const uint64_t per = p->scatter_group > 0 ? (uint64_t)p->scatter_group : 1;
  grid = std::max<uint64_t>(1, std::min<uint64_t>(grid, (total_chunks + per - 1) / per));
  if (w.chunk_desc) k_scatter<MODE, F32, true><<<(unsigned)grid, 256, 0, s>>>(p->view, w, total_chunks, per, counter);
  else k_scatter<MODE, F32, false><<<(unsigned)grid, 256, 0, s>>>(p->view, w, total_chunks, per, counter);
}

static void launch_scatter_any(ft_pool* p, int mode, bool f32, const WriteCall& w, uint64_t total_chunks, uint64_t max_ctas,
                               cudaStream_t s, ClaimCounter* cc) {
  if (mode == kTierAll) { if (f32) launch_scatter<kTierAll, true>(p, w, total_chunks, max_ctas, s, cc); else launch_scatter<kTierAll, false>(p, w, total_chunks, max_ctas, s, cc); }
  else if (mode == kTierDeviceOnly) { if (f32) launch_scatter<kTierDeviceOnly, true>(p, w, total_chunks, max_ctas, s, cc); else launch_scatter<kTierDeviceOnly, false>(p, w, total_chunks, max_ctas, s, cc); }
  else { if (f32) launch_scatter<kTierHostOnly, true>(p, w, total_chunks, max_ctas, s, cc); else launch_scatter<kTierHostOnly, false>(p, w, total_chunks, max_ctas, s, cc); }
}

// Host-tier pages of a producer call (bf16 source), page by page: source bytes -> shared -> host frame with
// bulk copies.  One warp per CTA; lanes translate 32 page ordinals at a time, lane 0 drives the ring; a
// handful of CTAs saturate the host link.
__global__ void __launch_bounds__(32) k_scatter_host_bulk(PoolView v, WriteCall c, uint64_t call_seq) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint64_t bars[kBulkStages];
  __shared__ uint64_t dst_q[kBulkStages];
  __shared__ uint32_t len_q[kBulkStages];
  const uint32_t lane = threadIdx.x;
  BulkRing ring;
  ring.init(smem, bars, dst_q, len_q, v.bulk_wait_ns, v.bulk_tx_slack);
  uint64_t item = 0;
  for (uint32_t q = 0; q < c.n; ++q) {
    const uint32_t sid = c.span_id[q];
    const uint64_t nbytes = (uint64_t)c.n_tokens[q] * v.row_bytes;
    const uint32_t npages = (uint32_t)((nbytes + v.page_bytes - 1) >> v.page_shift);
    const uint8_t* src_q = reinterpret_cast<const uint8_t*>(c.src[q]);
    for (uint32_t g = 0; g < npages; g += 32, ++item) {
      if (item % gridDim.x != blockIdx.x) continue;
      const uint32_t o = g + lane;
      uint64_t pte = 0, off;
      if (o < npages) pte = translate(v, span_page_gva(v, sid, o), &off);
      const bool host = (pte & kPteValid) && (pte & kPteHost);
      const uint32_t mask = __ballot_sync(0xFFFFFFFFu, host);
      for (uint32_t m = mask; m; m &= m - 1) {
        const int l = __ffs(m) - 1;
        const uint64_t p_l = __shfl_sync(0xFFFFFFFFu, pte, l);
        const uint64_t b0 = (uint64_t)(g + l) << v.page_shift;  // destination byte offset inside the span image
        const uint64_t len = min(v.page_bytes, nbytes - b0);
        uint8_t* dst = reinterpret_cast<uint8_t*>(p_l & ~kPteFlagMask);
        for (uint64_t x = 0; x < len; x += kBulkStageBytes)
          ring.push(src_q + b0 + x, dst + x, (uint32_t)min((uint64_t)kBulkStageBytes, len - x));
      }
    }
  }
  ring.drain();
  if (ring.lost && lane == 0) note_error(v, call_seq, FT_ERR_TIMEOUT, (blockIdx.x & 0xFFFFu) | (min(ring.stranded, 0xFFFFu) << 16));
}

int32_t scatter_set_carveout(int pct) {
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierAll, false, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierAll, false, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierAll, true, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierAll, true, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierDeviceOnly, false, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierDeviceOnly, false, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierDeviceOnly, true, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierDeviceOnly, true, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierHostOnly, false, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierHostOnly, false, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierHostOnly, true, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_scatter<kTierHostOnly, true, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  return FT_OK;
}

// The byte copy of a producer call, shared by pool_write_embeddings and its no-allocation variant: HBM-bound chunks on
// the caller's stream, host-bound chunks beside them on the producer side's second stream.
// The caller's arguments of a producer write, for the copy-engine path (which works from the host's page lists).
struct WriteArgs {
  uint32_t n;
  const uint32_t *slot, *span_idx, *n_tokens;
  const void* const* src;
};
bool host_tier_by_copy_engine(const ft_pool* p) {
  return p->host_dma == 1;
}
// bf16 sources into host-tier pages through the copy engine: one copy per run of pages that follow one another both
// in the span's image and in the host slab.  The pages come from the host's copy of the page lists (mirror_write ran).
static int32_t dma_write_host_pages(ft_pool* p, const WriteArgs& a, cudaStream_t s) {
  const uint64_t PS = p->cfg.page_bytes;
  const uint32_t S = p->cfg.max_spans_per_sample;
  uint8_t* base = static_cast<uint8_t*>(p->host_base);
  cudaError_t err = cudaSuccess;
  for (uint32_t q = 0; q < a.n; ++q) {
    const ft_span_mirror& m = p->spans[(uint64_t)a.slot[q] * S + a.span_idx[q]];
    const uint8_t* src = static_cast<const uint8_t*>(a.src[q]);
    for_each_host_run(p, m, (uint64_t)a.n_tokens[q] * p->view.row_bytes, [&](uint64_t off, uint64_t frame, uint64_t len) {
      if (err == cudaSuccess) err = cudaMemcpyAsync(base + frame * PS, src + off, len, cudaMemcpyDeviceToHost, s);
    });
  }
  if (err != cudaSuccess) return cuda_fail(err, "cudaMemcpyAsync(host-tier pages)");
  return FT_OK;
}

static int32_t launch_write_copies(ft_pool* p, const WriteCall& w, uint64_t total_chunks, bool f32, cudaStream_t st, ClaimCounter* cc,
                                   bool profile, const WriteArgs& args) {
  const ft_pool_config& c = p->cfg;
  auto launch = [&](int mode, cudaStream_t s) {
    const bool host_class = mode == kTierHostOnly || (mode == kTierAll && c.hbm_pages == 0);
    if (profile) prof_begin(p, host_class ? FT_K_SCATTER_HOST : FT_K_SCATTER_DEVICE, s);
    launch_scatter_any(p, mode, f32, w, total_chunks, host_class ? (uint64_t)p->host_store_ctas : ~0ull, s, cc);
    if (profile) prof_end(p, s);
    p->gpu_launches++;
  };
  if (c.host_pages == 0 || c.hbm_pages == 0) {
    launch(kTierAll, st);
  } else {
    FT_CUDA(cudaEventRecord(p->fork_ev[0], st));
    FT_CUDA(cudaStreamWaitEvent(p->side_stream[0], p->fork_ev[0], 0));
    if (profile) prof_begin(p, FT_K_SCATTER_HOST, p->side_stream[0]);
    // bf16 source: bulk-async copies through shared memory.  fp32 source: the cast needs the values in
    // registers, and stores to host memory are posted (no latency to hide), so a few vector-store CTAs do it
    if (f32) {
      launch_scatter<kTierHostOnly, true>(p, w, total_chunks, (uint64_t)p->host_store_ctas, p->side_stream[0], cc);
      p->gpu_launches++;
    } else if (host_tier_by_copy_engine(p)) {
      const int32_t rc = dma_write_host_pages(p, args, p->side_stream[0]);
      if (rc != FT_OK) return rc;
    } else {
      k_scatter_host_bulk<<<(unsigned)p->host_ctas, 32, kBulkSmemBytes, p->side_stream[0]>>>(p->view, w, status_seq(p));
      p->gpu_launches++;
    }
    if (profile) prof_end(p, p->side_stream[0]);
    FT_CUDA(cudaEventRecord(p->join_ev[0], p->side_stream[0]));
    launch(kTierDeviceOnly, st);
    FT_CUDA(cudaStreamWaitEvent(st, p->join_ev[0], 0));
  }
  FT_CUDA(cudaGetLastError());
  return FT_OK;
}

// ------------------------------------------------------------------------------------------
// K9: free
// ------------------------------------------------------------------------------------------
struct FreeCall {
  uint32_t n_spans, n_samples;
  const uint32_t* span_id;  // [n_spans] written spans, canonical order
  const uint32_t* slot;     // [n_samples]
  uint32_t* page_off;       // [n_spans+1]
  uint32_t* blk_off;        // [n_spans+1]
  uint32_t* tp_off;         // [n_samples+1]
  uint32_t* tails;          // [3] page ring, block ring, text ring tails before the pushes
};

__global__ void __launch_bounds__(1024) k_free_scan(PoolView v, FreeCall c) {
  // per span: list blocks to return, and pages to return unless the sample was imported (a peer owns them);
  // per sample: text pages to return, likewise
  uint64_t cp = 0, cb = 0, ct = 0;
  const uint32_t m = max(c.n_spans, c.n_samples);
  for (uint32_t base = 0; base < m; base += blockDim.x) {
    uint32_t i = base + threadIdx.x;
    uint64_t k = 0, nb = 0, nt = 0;
    if (i < c.n_spans) {
      const uint32_t sid = c.span_id[i];
      const uint32_t np = v.sp_npages[sid];
      nb = (np + kListBlock - 1) / kListBlock;
      k = (v.s_flags[sid / v.spans_per_sample] & 1) ? 0 : np;
    }
    if (i < c.n_samples && !(v.s_flags[c.slot[i]] & 1)) nt = (v.s_seq_len[c.slot[i]] + kTextPageIds - 1) / kTextPageIds;
    uint64_t tp, tb, tt;
    uint64_t ep = block_exclusive_scan(k, &tp);
    uint64_t eb = block_exclusive_scan(nb, &tb);
    uint64_t et = block_exclusive_scan(nt, &tt);
    if (i < c.n_spans) { c.page_off[i] = (uint32_t)(cp + ep); c.blk_off[i] = (uint32_t)(cb + eb); }
    if (i < c.n_samples) c.tp_off[i] = (uint32_t)(ct + et);
    cp += tp; cb += tb; ct += tt;
  }
  if (threadIdx.x == 0) {
    c.page_off[c.n_spans] = (uint32_t)cp; c.blk_off[c.n_spans] = (uint32_t)cb; c.tp_off[c.n_samples] = (uint32_t)ct;
    RingState s = *v.ring_state;
    c.tails[0] = (uint32_t)(((uint64_t)s.head + s.count) % v.ring_cap); s.count += (uint32_t)cp; *v.ring_state = s;
    s = *v.bring_state;
    c.tails[1] = (uint32_t)(((uint64_t)s.head + s.count) % v.bring_cap); s.count += (uint32_t)cb; *v.bring_state = s;
    s = *v.tring_state;
    c.tails[2] = (uint32_t)(((uint64_t)s.head + s.count) % v.tring_cap); s.count += (uint32_t)ct; *v.tring_state = s;
  }
}

__device__ __forceinline__ uint32_t last_le(const uint32_t* off, uint32_t n, uint32_t x) {
  uint32_t lo = 0, hi = n;  // largest i with off[i] <= x (off[0] = 0)
  while (hi - lo > 1) {
    uint32_t mid = (lo + hi) >> 1;
    if (off[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

// threads [0, P): one page each, pushed at the tail in canonical order; [P, P+B): one list block each;
// [P+B, P+B+T): one text page each
__global__ void __launch_bounds__(256) k_free_fill(PoolView v, FreeCall c, uint32_t total_pages, uint32_t total_blocks,
                                                  uint32_t total_text) {
  uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < total_pages) {
    // spans with no pages to return (imported) have equal consecutive offsets: last_le lands on the last of
    // a run of equal offsets, which is the span that owns entry t
    const uint32_t q = last_le(c.page_off, c.n_spans, t), o = t - c.page_off[q], sid = c.span_id[q];
    v.ring[(c.tails[0] + t) % v.ring_cap] = global_page_of(v, span_page_gva(v, sid, o));
    return;
  }
  t -= total_pages;
  if (t < total_blocks) {
    const uint32_t q = last_le(c.blk_off, c.n_spans, t), b = t - c.blk_off[q], sid = c.span_id[q];
    v.bring[(c.tails[1] + t) % v.bring_cap] = v.sp_blocks[(uint64_t)sid * v.blocks_per_span + b];
    return;
  }
  t -= total_blocks;
  if (t < total_text) {
    const uint32_t i = last_le(c.tp_off, c.n_samples, t), k = t - c.tp_off[i], slot = c.slot[i];
    const uint64_t g = v.s_text_pages[(uint64_t)slot * v.text_pages_per_sample + k];
    v.tring[(c.tails[2] + t) % v.tring_cap] = (uint32_t)((g - v.text_gva_base) / FT_TEXT_PAGE_BYTES);
  }
}

__global__ void k_free_clear(PoolView v, FreeCall c) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < c.n_spans) v.sp_npages[c.span_id[i]] = 0;
  if (i < c.n_samples) { v.s_seq_len[c.slot[i]] = 0; v.s_n_spans[c.slot[i]] = 0; v.s_flags[c.slot[i]] = 0; }
}

__global__ void k_debug_translate(PoolView v, const uint64_t* gva, uint32_t n, uint32_t* kind, uint64_t* frame,
                                  uint64_t* offset, int32_t* status, const uint64_t* bases /* [world][3] */) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint64_t off = 0;
  const uint64_t pte = translate(v, gva[i], &off);
  if (!(pte & kPteValid)) { status[i] = FT_ERR_BAD_GVA; kind[i] = 0; frame[i] = 0; offset[i] = 0; return; }
  // the owning process, to express the frame as an index into that process's slab
  uint64_t proc = 0;
  for (int t = 0; t < 2; ++t) {
    const uint64_t d = gva[i] - v.region_start[t];
    if (d < v.region_bytes) proc = d / v.max_size;
  }
  const uint64_t addr = pte & ~kPteFlagMask;
  status[i] = FT_OK;
  offset[i] = off;
  if (pte & kPteText) { kind[i] = 2; frame[i] = (addr - bases[3 * proc + 2]) / FT_TEXT_PAGE_BYTES; }
  else if (pte & kPteHost) { kind[i] = 1; frame[i] = (addr - bases[3 * proc + 1]) >> v.page_shift; }
  else { kind[i] = 0; frame[i] = (addr - bases[3 * proc]) >> v.page_shift; }
}

static inline uint64_t pages_for_tokens(const ft_pool* p, uint64_t n_tokens) {
  const uint64_t bytes = n_tokens * 2ull * p->cfg.hidden;
  return (bytes + p->cfg.page_bytes - 1) / p->cfg.page_bytes;
}

}  // namespace ft

using namespace ft;

// ==========================================================================================
// C ABI
// ==========================================================================================
extern "C" __attribute__((visibility("default"))) const char* flowpool_last_cuda_error(void) { return ft::g_last_error; }

extern "C" __attribute__((visibility("default"))) int32_t pool_destroy(ft_pool* p) {
  if (!p) return FT_ERR_INVALID_ARG;
  cudaSetDevice(p->device);
  cudaDeviceSynchronize();
  for (ft_call_ctx* ring : {p->ctx[0], p->ctx[1]}) for (int i = 0; i < kCallCtx; ++i) {
    ft_call_ctx& c = ring[i];
    if (c.h) cudaFreeHost(c.h);
    if (c.d) cudaFree(c.d);
    if (c.ev_up) cudaEventDestroy(c.ev_up);
    if (c.ev_done) cudaEventDestroy(c.ev_done);
  }
  ft::pool_registry_remove(p);
  for (auto& b : p->plan_cache) { if (b.d) cudaFree(b.d); if (b.ev) cudaEventDestroy(b.ev); }
  if (p->plan_pinned) cudaFreeHost(p->plan_pinned);
  if (p->meta) cudaStreamDestroy(p->meta);
  if (p->ev_meta) cudaEventDestroy(p->ev_meta);
  if (p->ev_in) cudaEventDestroy(p->ev_in);
  if (p->ev_ids) cudaEventDestroy(p->ev_ids);
  if (p->ev_noalloc) cudaEventDestroy(p->ev_noalloc);
  for (void* a : p->peer_allocs) cudaFree(a);
  if (p->d_meta) cudaFree(p->d_meta);
  if (p->d_text) cudaFree(p->d_text);
  if (p->own_hbm && p->hbm_base) cudaFree(p->hbm_base);
  if (p->own_host && p->host_base) cudaFreeHost(p->host_base);
  for (int a = 0; a < 3; ++a) {
    if (p->side_stream[a]) cudaStreamDestroy(p->side_stream[a]);
    if (p->fork_ev[a]) cudaEventDestroy(p->fork_ev[a]);
    if (p->join_ev[a]) cudaEventDestroy(p->join_ev[a]);
  }
  if (p->ev_producer) cudaEventDestroy(p->ev_producer);
  if (p->ev_consumer) cudaEventDestroy(p->ev_consumer);
  delete p;
  cudaGetLastError();
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_create(const ft_pool_config* cfg_in, void* hbm_base, void* host_base, ft_pool** out) {
  if (!cfg_in || !out) return FT_ERR_INVALID_ARG;
  ft_pool_config c = *cfg_in;
  if (c.gva_hbm_start == 0) c.gva_hbm_start = 1ull << 44;
  if (c.gva_host_start == 0) c.gva_host_start = 1ull << 45;
  if (c.max_size == 0) c.max_size = 1ull << 40;
  if (c.world_size == 0) c.world_size = 1;
  const uint64_t PS = c.page_bytes;
  if (PS < 4096 || PS > (2u << 20) || (PS & (PS - 1))) return FT_ERR_INVALID_ARG;
  if (c.hidden == 0 || c.hidden % 8) return FT_ERR_INVALID_ARG;
  if (c.hbm_pages + c.host_pages == 0) return FT_ERR_INVALID_ARG;
  if (c.hbm_pages + c.host_pages > 0xFFFFFFFFull) return FT_ERR_INVALID_ARG;
  if (c.rank >= c.world_size) return FT_ERR_INVALID_ARG;
  if (c.max_samples == 0 || c.max_seq_len == 0) return FT_ERR_INVALID_ARG;
  if (c.max_spans_per_sample == 0) c.max_spans_per_sample = 1;
  if (c.max_pages_per_span == 0) c.max_pages_per_span = 1;
  const uint64_t n_text = (c.max_text_tokens + kTextPageIds - 1) / kTextPageIds;
  if (c.hbm_pages * PS + n_text * FT_TEXT_PAGE_BYTES > c.max_size) return FT_ERR_INVALID_ARG;
  if (c.host_pages * PS > c.max_size) return FT_ERR_INVALID_ARG;
  const uint64_t region = (uint64_t)c.world_size * c.max_size;
  if (c.gva_hbm_start + region < c.gva_hbm_start || c.gva_host_start + region < c.gva_host_start) return FT_ERR_INVALID_ARG;
  if (c.gva_hbm_start < c.gva_host_start + region && c.gva_host_start < c.gva_hbm_start + region) return FT_ERR_INVALID_ARG;
  if (hbm_base && (reinterpret_cast<uintptr_t>(hbm_base) & 255)) return FT_ERR_INVALID_ARG;
  if (host_base && (reinterpret_cast<uintptr_t>(host_base) & 255)) return FT_ERR_INVALID_ARG;

  ft_pool* p = new ft_pool();
  p->cfg = c;
  int32_t rc = FT_OK;
#define CK(call)                                                                          \
  do {                                                                                    \
    cudaError_t e__ = (call);                                                             \
    if (e__ != cudaSuccess) { rc = ft::cuda_fail(e__, #call); pool_destroy(p); return rc; } \
  } while (0)
  CK(cudaGetDevice(&p->device));
  CK(cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, p->device));
  for (int a = 0; a < 3; ++a) {
    CK(cudaStreamCreateWithFlags(&p->side_stream[a], cudaStreamNonBlocking));
    CK(cudaEventCreateWithFlags(&p->fork_ev[a], cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&p->join_ev[a], cudaEventDisableTiming));
  }
  CK(cudaEventCreateWithFlags(&p->ev_producer, cudaEventDisableTiming));
  CK(cudaEventCreateWithFlags(&p->ev_consumer, cudaEventDisableTiming));
  CK(cudaStreamCreateWithFlags(&p->meta, cudaStreamNonBlocking));
  CK(cudaEventCreateWithFlags(&p->ev_meta, cudaEventDisableTiming));
  CK(cudaEventCreateWithFlags(&p->ev_in, cudaEventDisableTiming));
  CK(cudaEventCreateWithFlags(&p->ev_ids, cudaEventDisableTiming));
  CK(cudaEventCreateWithFlags(&p->ev_noalloc, cudaEventDisableTiming));
  // every call context starts with 64 KiB of pinned staging and 256 KiB of device scratch (enough for calls of a few
  // thousand spans), so that no call of ordinary size allocates; larger calls grow their context on demand
  for (int side = 0; side < 2; ++side) for (int i = 0; i < kCallCtx; ++i) {
    ft_call_ctx& cx = p->ctx[side][i];
    CK(cudaEventCreateWithFlags(&cx.ev_up, cudaEventDisableTiming));
    CK(cudaEventCreateWithFlags(&cx.ev_done, cudaEventDisableTiming));
    CK(cudaHostAlloc(&cx.h, 1 << 16, cudaHostAllocMapped));
    CK(cudaHostGetDevicePointer(&cx.hd, cx.h, 0));
    cx.hcap = 1 << 16;
    CK(cudaMalloc(&cx.d, 1 << 18));
    cx.dcap = 1 << 18;
  }
  p->noalloc_blob.resize(16 * (size_t)FT_NOALLOC_MAX_SPANS + 256);
  // per-device kernel set-up: shared-memory opt-ins and occupancy of the data kernels
  CK(cudaFuncSetAttribute(k_scatter_host_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBulkSmemBytes));
  {
    auto occ = [](auto kernel) { int v = 0; return cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, kernel, 256, 0) == cudaSuccess && v > 0 ? v : 1; };
    p->occ_scatter[kTierAll][0] = std::min(occ(k_scatter<kTierAll, false, false>), occ(k_scatter<kTierAll, false, true>)); p->occ_scatter[kTierAll][1] = std::min(occ(k_scatter<kTierAll, true, false>), occ(k_scatter<kTierAll, true, true>));
    p->occ_scatter[kTierDeviceOnly][0] = std::min(occ(k_scatter<kTierDeviceOnly, false, false>), occ(k_scatter<kTierDeviceOnly, false, true>)); p->occ_scatter[kTierDeviceOnly][1] = std::min(occ(k_scatter<kTierDeviceOnly, true, false>), occ(k_scatter<kTierDeviceOnly, true, true>));
    p->occ_scatter[kTierHostOnly][0] = std::min(occ(k_scatter<kTierHostOnly, false, false>), occ(k_scatter<kTierHostOnly, false, true>)); p->occ_scatter[kTierHostOnly][1] = std::min(occ(k_scatter<kTierHostOnly, true, false>), occ(k_scatter<kTierHostOnly, true, true>));
  }
  // the scatter kernel's shared-memory split (see ft_tuning.scatter_smem_carveout): small but stated, so that metadata
  // kernels and the packing kernel can start on SMs that hold its CTAs
  if ((rc = scatter_set_carveout(p->scatter_smem_carveout)) != FT_OK) { pool_destroy(p); return rc; }
  if ((rc = gather_device_setup(p)) != FT_OK || (rc = plan_device_setup(p)) != FT_OK) { pool_destroy(p); return rc; }

  const uint64_t P = c.hbm_pages + c.host_pages;
  const uint32_t S = c.max_spans_per_sample;
  const uint32_t TPS = (c.max_seq_len + kTextPageIds - 1) / kTextPageIds;
  const uint32_t MB = (c.max_pages_per_span + kListBlock - 1) / kListBlock;
  const uint64_t span_ids = (uint64_t)c.max_samples * S;
  // list blocks: one per 64 pages plus at most one partial block per live span; imported samples bring pages that
  // are not local, budgeted by max_imported_pages
  const uint64_t imp = c.max_imported_pages;
  const uint64_t NB = (P + imp + kListBlock - 1) / kListBlock + std::min<uint64_t>(span_ids, P + imp) + 1;
  if (NB > 0xFFFFFFFFull || span_ids > 0xFFFFFFFFull) { pool_destroy(p); return FT_ERR_INVALID_ARG; }

  // backing memory
  if (c.hbm_pages) {
    if (hbm_base) p->hbm_base = hbm_base;
    else { CK(cudaMalloc(&p->hbm_base, c.hbm_pages * PS)); p->own_hbm = true; }
  }
  if (c.host_pages) {
    if (host_base) p->host_base = host_base;
    else { CK(cudaHostAlloc(&p->host_base, c.host_pages * PS, cudaHostAllocMapped | cudaHostAllocPortable)); p->own_host = true; }
    cudaError_t e = cudaHostGetDevicePointer(&p->host_dev, p->host_base, 0);
    if (e != cudaSuccess) { ft::cuda_fail(e, "cudaHostGetDevicePointer(host_base)"); pool_destroy(p); return host_base ? FT_ERR_INVALID_ARG : FT_ERR_CUDA; }
  }
  CK(cudaMalloc(&p->d_text, std::max<uint64_t>(n_text, 1) * FT_TEXT_PAGE_BYTES));

  // metadata block
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t o_pte_hbm = take(c.hbm_pages * 8), o_pte_host = take(c.host_pages * 8), o_pte_text = take(n_text * 8);
  const size_t o_ring = take(P * 4), o_tring = take(n_text * 4), o_bring = take(NB * 4);
  // status word, then two claim counters per call context (zero at rest)
  const size_t o_states = take(3 * sizeof(RingState)), o_status = take(64 + (size_t)2 * kCallCtx * 2 * sizeof(ClaimCounter));
  const size_t o_seq = take((size_t)c.max_samples * 4), o_nsp = take((size_t)c.max_samples * 4);
  const size_t o_stp = take((size_t)c.max_samples * TPS * 8), o_sfl = take((size_t)c.max_samples * 4);
  const size_t o_peers = take((size_t)c.world_size * sizeof(PeerTables));
  const size_t o_pos = take(span_ids * 4), o_tok = take(span_ids * 4), o_npg = take(span_ids * 4);
  const size_t o_blk = take(span_ids * MB * 4), o_lst = take(NB * kListBlock * 8);
  const size_t o_grid = take(span_ids * sizeof(uint4));
  CK(cudaMalloc(&p->d_meta, off));
  CK(cudaMemset(p->d_meta, 0, off));
  uint8_t* m = static_cast<uint8_t*>(p->d_meta);

  PoolView& v = p->view;
  v.region_start[0] = c.gva_hbm_start; v.region_start[1] = c.gva_host_start;
  v.region_bytes = region; v.max_size = c.max_size;
  v.seg_base[0] = c.gva_hbm_start + (uint64_t)c.rank * c.max_size;
  v.seg_base[1] = c.gva_host_start + (uint64_t)c.rank * c.max_size;
  v.text_gva_base = v.seg_base[0] + c.hbm_pages * PS;
  v.rank = c.rank;
  v.page_shift = 0; while ((1ull << v.page_shift) < PS) ++v.page_shift;
  v.page_bytes = PS; v.hbm_pages = c.hbm_pages; v.host_pages = c.host_pages; v.text_pages = n_text;
  v.hidden = c.hidden; v.row_bytes = 2 * c.hidden; v.placeholder_id = c.placeholder_id;
  v.max_samples = c.max_samples; v.spans_per_sample = S; v.text_pages_per_sample = TPS; v.blocks_per_span = MB;
  v.pte_hbm = reinterpret_cast<uint64_t*>(m + o_pte_hbm);
  v.pte_host = reinterpret_cast<uint64_t*>(m + o_pte_host);
  v.pte_text = reinterpret_cast<uint64_t*>(m + o_pte_text);
  v.ring = reinterpret_cast<uint32_t*>(m + o_ring); v.ring_cap = (uint32_t)P;
  v.tring = reinterpret_cast<uint32_t*>(m + o_tring); v.tring_cap = (uint32_t)std::max<uint64_t>(n_text, 1);
  v.bring = reinterpret_cast<uint32_t*>(m + o_bring); v.bring_cap = (uint32_t)NB;
  RingState* st = reinterpret_cast<RingState*>(m + o_states);
  v.ring_state = st; v.tring_state = st + 1; v.bring_state = st + 2;
  v.status = reinterpret_cast<unsigned long long*>(m + o_status);
  v.bulk_wait_ns = kBulkWaitLimitNs;
  v.bulk_tx_slack = 0;
  for (int i = 0; i < 2 * kCallCtx; ++i) p->ctx[i / kCallCtx][i % kCallCtx].counters = reinterpret_cast<ClaimCounter*>(m + o_status + 64) + 2 * i;
  v.s_seq_len = reinterpret_cast<uint32_t*>(m + o_seq); v.s_n_spans = reinterpret_cast<uint32_t*>(m + o_nsp);
  v.s_text_pages = reinterpret_cast<uint64_t*>(m + o_stp);
  v.s_flags = reinterpret_cast<uint32_t*>(m + o_sfl);
  v.peers = reinterpret_cast<PeerTables*>(m + o_peers);
  v.world_size = c.world_size;
  v.sp_pos = reinterpret_cast<uint32_t*>(m + o_pos); v.sp_tokens = reinterpret_cast<uint32_t*>(m + o_tok);
  v.sp_npages = reinterpret_cast<uint32_t*>(m + o_npg); v.sp_blocks = reinterpret_cast<uint32_t*>(m + o_blk);
  v.list_blocks = reinterpret_cast<uint64_t*>(m + o_lst);
  v.sp_grid = reinterpret_cast<uint4*>(m + o_grid);

  // binding (identity or seeded permutation per tier) and the initial ring order are made on the host, once
  std::vector<uint32_t> bind_h(c.hbm_pages), bind_d(c.host_pages), ring(P);
  for (uint64_t k = 0; k < c.hbm_pages; ++k) bind_h[k] = (uint32_t)k;
  for (uint64_t k = 0; k < c.host_pages; ++k) bind_d[k] = (uint32_t)k;
  for (uint64_t k = 0; k < P; ++k) ring[k] = (uint32_t)k;
  if (c.bind_order == FT_BIND_PERMUTED) { seeded_shuffle(bind_h, c.bind_seed); seeded_shuffle(bind_d, c.bind_seed + 1); }
  if (c.ring_order == FT_RING_SHUFFLED) seeded_shuffle(ring, c.ring_seed);
  uint32_t* d_tmp = nullptr;
  CK(cudaMalloc(&d_tmp, std::max<uint64_t>(P, 1) * 4));
  auto blocks = [](uint64_t n) { return (unsigned)((n + 255) / 256); };
  if (c.hbm_pages) {
    CK(cudaMemcpy(d_tmp, bind_h.data(), c.hbm_pages * 4, cudaMemcpyHostToDevice));
    k_page_table_init<<<blocks(c.hbm_pages), 256>>>(const_cast<uint64_t*>(v.pte_hbm), d_tmp, c.hbm_pages,
                                                   reinterpret_cast<uint64_t>(p->hbm_base), PS, kPteValid);
    CK(cudaDeviceSynchronize());
  }
  if (c.host_pages) {
    CK(cudaMemcpy(d_tmp, bind_d.data(), c.host_pages * 4, cudaMemcpyHostToDevice));
    k_page_table_init<<<blocks(c.host_pages), 256>>>(const_cast<uint64_t*>(v.pte_host), d_tmp, c.host_pages,
                                                    reinterpret_cast<uint64_t>(p->host_dev), PS, kPteValid | kPteHost);
    CK(cudaDeviceSynchronize());
  }
  if (n_text) {
    k_page_table_init<<<blocks(n_text), 256>>>(const_cast<uint64_t*>(v.pte_text), nullptr, n_text,
                                              reinterpret_cast<uint64_t>(p->d_text), FT_TEXT_PAGE_BYTES, kPteValid | kPteText);
    k_iota<<<blocks(n_text), 256>>>(v.tring, n_text);
  }
  k_iota<<<blocks(NB), 256>>>(v.bring, NB);
  CK(cudaMemcpy(v.ring, ring.data(), P * 4, cudaMemcpyHostToDevice));
  RingState init[3] = {{0, (uint32_t)P}, {0, (uint32_t)n_text}, {0, (uint32_t)NB}};
  CK(cudaMemcpy(st, init, sizeof(init), cudaMemcpyHostToDevice));
  CK(cudaMemset(v.status, 0xFF, 8));
  {  // this process's own entry of the collected page tables
    PeerTables self{v.pte_hbm, v.pte_host, v.pte_text, v.hbm_pages, v.host_pages, v.text_pages};
    CK(cudaMemcpy(const_cast<PeerTables*>(v.peers) + c.rank, &self, sizeof(self), cudaMemcpyHostToDevice));
  }
  p->peer_imported.assign(c.world_size, 0);
  p->peer_imported[c.rank] = 1;
  p->peer_bases.assign(c.world_size, {0, 0, 0});
  p->peer_bases[c.rank] = {reinterpret_cast<uint64_t>(p->hbm_base), reinterpret_cast<uint64_t>(p->host_dev), reinterpret_cast<uint64_t>(p->d_text)};
  CK(cudaDeviceSynchronize());
  CK(cudaFree(d_tmp));
  p->bind_hbm = bind_h; p->bind_host = bind_d;
  p->h_ring = ring; p->h_ring_head = 0; p->h_ring_count = P;
  p->h_page_next.assign(P, kNone);
  p->gpu_launches += 5;
#undef CK
  p->slots.resize(c.max_samples);
  p->spans.resize(span_ids);
  p->free_pages = P; p->free_text_pages = n_text; p->free_blocks = NB;
  ft::pool_registry_add(p);
  *out = p;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_register_samples(ft_pool* p, uint32_t n, const uint32_t* slot, const uint32_t* seq_len,
                                         const uint32_t* n_spans, const uint32_t* span_pos,
                                         const uint32_t* span_tokens, const int32_t* input_ids, void* stream) {
  if (!p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (n == 0) return FT_OK;
  if (!slot || !seq_len || !n_spans || !input_ids) return FT_ERR_INVALID_ARG;
  const ft_pool_config& c = p->cfg;
  uint64_t text_need = 0, sp = 0;
  std::vector<uint8_t> seen(c.max_samples, 0);
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= c.max_samples) return FT_ERR_INVALID_ARG;
    if (p->slots[slot[i]].state != FT_SLOT_FREE || seen[slot[i]]) return FT_ERR_SLOT_IN_USE;
    seen[slot[i]] = 1;
    if (seq_len[i] == 0) return FT_ERR_INVALID_ARG;
    if (seq_len[i] > c.max_seq_len) return FT_ERR_CAPACITY;
    if (n_spans[i] > c.max_spans_per_sample) return FT_ERR_CAPACITY;
    if (n_spans[i] && (!span_pos || !span_tokens)) return FT_ERR_INVALID_ARG;
    uint64_t prev_end = 0;
    for (uint32_t j = 0; j < n_spans[i]; ++j, ++sp) {
      if (span_tokens[sp] == 0) return FT_ERR_INVALID_ARG;
      if ((uint64_t)span_pos[sp] + span_tokens[sp] > seq_len[i]) return FT_ERR_INVALID_ARG;
      if (span_pos[sp] < prev_end) return FT_ERR_INVALID_ARG;
      prev_end = (uint64_t)span_pos[sp] + span_tokens[sp];
      if (pages_for_tokens(p, span_tokens[sp]) > c.max_pages_per_span) return FT_ERR_CAPACITY;
    }
    text_need += (seq_len[i] + kTextPageIds - 1) / kTextPageIds;
  }
  if (text_need > p->free_text_pages) return FT_ERR_CAPACITY;
  const uint64_t total_spans = sp;

  // descriptor blob: [ids_off u64 (n+1)] [slot][seq_len][n_spans][span_begin (n+1)][span_pos][span_tok]
  const size_t o_idsoff = 0, o_slot = align_up((size_t)(n + 1) * 8, 16);
  const size_t o_len = o_slot + (size_t)n * 4, o_nsp = o_len + (size_t)n * 4, o_sb = o_nsp + (size_t)n * 4;
  const size_t o_pos = o_sb + (size_t)(n + 1) * 4, o_tok = o_pos + total_spans * 4;
  const size_t blob_bytes = align_up(o_tok + total_spans * 4, 256);
  const size_t o_tpoff = blob_bytes, o_head = align_up(o_tpoff + (size_t)(n + 1) * 4, 16);
  const size_t o_pgdst = o_head + 16, o_pgs = o_pgdst + (size_t)text_need * 8;
  const size_t total_bytes = o_pgs + (size_t)text_need * 4;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ft_call_ctx* cx = nullptr;
  int32_t rc = ctx_acquire(p, 0, blob_bytes, total_bytes, &cx);
  if (rc != FT_OK) return rc;
  uint8_t* hb = static_cast<uint8_t*>(cx->h);
  uint64_t* ids_off = reinterpret_cast<uint64_t*>(hb + o_idsoff);
  uint32_t* sb = reinterpret_cast<uint32_t*>(hb + o_sb);
  ids_off[0] = 0; sb[0] = 0;
  for (uint32_t i = 0; i < n; ++i) { ids_off[i + 1] = ids_off[i] + seq_len[i]; sb[i + 1] = sb[i] + n_spans[i]; }
  memcpy(hb + o_slot, slot, (size_t)n * 4);
  memcpy(hb + o_len, seq_len, (size_t)n * 4);
  memcpy(hb + o_nsp, n_spans, (size_t)n * 4);
  if (total_spans) {
    memcpy(hb + o_pos, span_pos, total_spans * 4);
    memcpy(hb + o_tok, span_tokens, total_spans * 4);
  }
  if ((rc = ctx_upload(p, cx, blob_bytes)) != FT_OK) return rc;
  uint8_t* db = static_cast<uint8_t*>(cx->d);
  RegisterCall rcall;
  rcall.n = n;
  rcall.ids_off = reinterpret_cast<uint64_t*>(db + o_idsoff);
  rcall.slot = reinterpret_cast<uint32_t*>(db + o_slot);
  rcall.seq_len = reinterpret_cast<uint32_t*>(db + o_len);
  rcall.n_spans = reinterpret_cast<uint32_t*>(db + o_nsp);
  rcall.span_begin = reinterpret_cast<uint32_t*>(db + o_sb);
  rcall.span_pos = reinterpret_cast<uint32_t*>(db + o_pos);
  rcall.span_tok = reinterpret_cast<uint32_t*>(db + o_tok);
  rcall.ids = input_ids;
  rcall.tp_off = reinterpret_cast<uint32_t*>(db + o_tpoff);
  rcall.head = reinterpret_cast<uint32_t*>(db + o_head);
  rcall.pg_dst = reinterpret_cast<uint64_t*>(db + o_pgdst);
  rcall.pg_sample = reinterpret_cast<uint32_t*>(db + o_pgs);
  rcall.call_seq = status_seq(p);
  // tables and the text-page pops on the metadata stream; the ids themselves (the caller's data) on the caller's
  k_register_scan<<<1, scan_threads(n), 0, p->meta>>>(p->view, rcall);
  if ((rc = meta_to(p, st)) != FT_OK) return rc;
  k_register_ids<<<(unsigned)text_need, 256, 0, st>>>(p->view, rcall);
  FT_CUDA(cudaGetLastError());
  FT_CUDA(cudaEventRecord(p->ev_ids, st));
  p->have_ids_ev = true;
  if ((rc = ctx_release(p, cx, st)) != FT_OK) return rc;
  p->gpu_launches += 2;

  // host mirror
  sp = 0;
  for (uint32_t i = 0; i < n; ++i) {
    ft_slot_mirror& s = p->slots[slot[i]];
    s.state = n_spans[i] == 0 ? FT_SLOT_READY : FT_SLOT_REGISTERED;
    if (s.state == FT_SLOT_READY) ready_push(p, slot[i]);  // text only: paired at once
    s.seq_len = seq_len[i]; s.n_spans = n_spans[i]; s.spans_written = 0;
    s.n_text_pages = (seq_len[i] + kTextPageIds - 1) / kTextPageIds;
    for (uint32_t j = 0; j < n_spans[i]; ++j, ++sp) {
      ft_span_mirror& m = p->spans[(uint64_t)slot[i] * c.max_spans_per_sample + j];
      m.pos = span_pos[sp]; m.tokens = span_tokens[sp]; m.npages = 0; m.written = false;
      m.grid[0] = m.grid[1] = m.grid[2] = 0;
    }
    p->live_samples++; p->live_spans += n_spans[i];
  }
  p->free_text_pages -= text_need;
  return end_producer(p, st);
}

namespace ft {
// Argument and state checks of a producer write, shared by both entry points (same codes, same order).  On success
// the call's totals are in `t` and, when `b_*` are given, the descriptors in the caller's staging arrays.
struct WriteTotals {
  uint64_t need = 0, need_blocks = 0, total_chunks = 0, bytes_total = 0;
  uint32_t chunk_shift = 16;  // the copy's work unit for this call
};
// The copy's work unit when the tuning leaves it open: the smaller the chunk, the shorter the kernel's last wave (a
// producer call of 0.7 GB streams at 6.3 TB/s with 64 KiB chunks and at 6.5 TB/s with 16 KiB chunks), as long as the
// per-chunk records stay a small table; `fine` = the caller can hold such records.
static uint32_t auto_chunk_shift(const uint64_t chunks_at[3], bool fine) {
  if (fine)
    for (int i = 0; i < 2; ++i)
      if (chunks_at[i] <= (1u << 17)) return 14 + i;
  return 16;
}
static int32_t check_write(ft_pool* p, uint32_t n, const uint32_t* slot, const uint32_t* span_idx, const uint32_t* n_tokens,
                           const void* const* src, WriteTotals* t, bool fine_chunks) {
  const ft_pool_config& c = p->cfg;
  const uint32_t S = c.max_spans_per_sample;
  uint64_t chunks_at[3] = {0, 0, 0};  // with 16, 32 and 64 KiB chunks
  uint64_t chunks_fixed = 0;
  for (uint32_t q = 0; q < n; ++q) {
    if (slot[q] >= c.max_samples) return FT_ERR_INVALID_ARG;
    const ft_slot_mirror& s = p->slots[slot[q]];
    if (s.state == FT_SLOT_FREE) return FT_ERR_UNKNOWN_SAMPLE;
    if (span_idx[q] >= s.n_spans) return FT_ERR_INVALID_ARG;
    ft_span_mirror& m = p->spans[(uint64_t)slot[q] * S + span_idx[q]];
    if (n_tokens[q] != m.tokens) return FT_ERR_INVALID_ARG;
    if (!src[q] || (reinterpret_cast<uintptr_t>(src[q]) & 15)) return FT_ERR_INVALID_ARG;
    if (m.written || m.named == p->call_seq) return FT_ERR_ALREADY_WRITTEN;  // written before, or named twice in this call
    m.named = p->call_seq;
    const uint64_t k = pages_for_tokens(p, n_tokens[q]);
    t->need += k; t->need_blocks += (k + kListBlock - 1) / kListBlock;
    const uint64_t bytes = (uint64_t)n_tokens[q] * p->view.row_bytes;
    for (int i = 0; i < 3; ++i) chunks_at[i] += (bytes + (1ull << (14 + i)) - 1) >> (14 + i);
    if (p->chunk_shift) chunks_fixed += (bytes + (1ull << p->chunk_shift) - 1) >> p->chunk_shift;
    t->bytes_total += bytes;
  }
  if (p->chunk_shift) {
    t->chunk_shift = (uint32_t)p->chunk_shift; t->total_chunks = chunks_fixed;
  } else {
    t->chunk_shift = auto_chunk_shift(chunks_at, fine_chunks && c.page_bytes >= (1u << 14));
    t->total_chunks = chunks_at[t->chunk_shift - 14];
  }
  if (t->need > p->free_pages) return FT_ERR_POOL_EXHAUSTED;
  if (t->need_blocks > p->free_blocks) return FT_ERR_CAPACITY;
  if (t->need > 0xFFFFFFFFull) return FT_ERR_INVALID_ARG;
  return FT_OK;
}

static void mirror_write(ft_pool* p, uint32_t n, const uint32_t* slot, const uint32_t* span_idx, const uint32_t* n_tokens,
                         const WriteTotals& t, bool f32) {
  const uint32_t S = p->cfg.max_spans_per_sample;
  for (uint32_t q = 0; q < n; ++q) {
    ft_slot_mirror& s = p->slots[slot[q]];
    ft_span_mirror& m = p->spans[(uint64_t)slot[q] * S + span_idx[q]];
    m.written = true; m.npages = (uint32_t)pages_for_tokens(p, n_tokens[q]);
    uint32_t prev = kNone;  // the ring's next entries, as k_alloc_fill takes them, chained in order
    for (uint32_t k = 0; k < m.npages; ++k) {
      const uint32_t g = p->h_ring[p->h_ring_head];
      p->h_ring_head = (p->h_ring_head + 1) % p->h_ring.size();
      if (prev == kNone) m.first_page = g; else p->h_page_next[prev] = g;
      prev = g;
    }
    m.owned_pages = m.npages;
    p->h_ring_count -= m.npages;
    if (++s.spans_written == s.n_spans) { s.state = FT_SLOT_READY; ready_push(p, slot[q]); }
  }
  p->free_pages -= t.need; p->free_blocks -= t.need_blocks;
  p->bytes_written += t.bytes_total * (f32 ? 3 : 2);
}
}  // namespace ft

extern "C" __attribute__((visibility("default"))) int32_t pool_write_embeddings(ft_pool* p, uint32_t n, const uint32_t* slot, const uint32_t* span_idx,
                                         const uint32_t* n_tokens, const void* const* src, uint32_t src_dtype,
                                         void* stream) {
  if (!p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (src_dtype != FT_BF16 && src_dtype != FT_F32) return FT_ERR_INVALID_ARG;
  if (n == 0) return FT_OK;
  if (!slot || !span_idx || !n_tokens || !src) return FT_ERR_INVALID_ARG;
  const uint32_t S = p->cfg.max_spans_per_sample;
  WriteTotals t;
  int32_t rc = check_write(p, n, slot, span_idx, n_tokens, src, &t, true);
  if (rc != FT_OK) return rc;
  const uint64_t need = t.need, total_chunks = t.total_chunks;

  // blob: [src u64 n][span_id n][n_tokens n] ; outputs: page_off, blk_off (n+1), chunk_off u64 (n+1), heads
  const size_t o_src = 0, o_sid = (size_t)n * 8, o_ntk = o_sid + (size_t)n * 4;
  const size_t blob_bytes = align_up(o_ntk + (size_t)n * 4, 256);
  const size_t o_choff = blob_bytes, o_poff = align_up(o_choff + (size_t)(n + 1) * 8, 16);
  const size_t o_boff = o_poff + (size_t)(n + 1) * 4, o_heads = align_up(o_boff + (size_t)(n + 1) * 4, 16);
  const size_t o_cspan = o_heads + 16;
  // chunk records for the copy kernel where a chunk cannot straddle a page (pages at least a chunk long)
  const bool with_desc = p->cfg.page_bytes >= (1ull << t.chunk_shift);
  const size_t o_cdesc = align_up(o_cspan + total_chunks * 4, 16);
  const size_t total_bytes = o_cdesc + (with_desc ? total_chunks * sizeof(ChunkDesc) : 0);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ft_call_ctx* cx = nullptr;
  if ((rc = ctx_acquire(p, 0, blob_bytes, total_bytes, &cx)) != FT_OK) return rc;
  uint8_t* hb = static_cast<uint8_t*>(cx->h);
  for (uint32_t q = 0; q < n; ++q) {
    reinterpret_cast<uint64_t*>(hb + o_src)[q] = reinterpret_cast<uint64_t>(src[q]);
    reinterpret_cast<uint32_t*>(hb + o_sid)[q] = slot[q] * S + span_idx[q];
  }
  memcpy(hb + o_ntk, n_tokens, (size_t)n * 4);
  if ((rc = ctx_upload(p, cx, blob_bytes)) != FT_OK) return rc;
  uint8_t* db = static_cast<uint8_t*>(cx->d);
  WriteCall w;
  w.n = n;
  w.src = reinterpret_cast<uint64_t*>(db + o_src);
  w.span_id = reinterpret_cast<uint32_t*>(db + o_sid);
  w.n_tokens = reinterpret_cast<uint32_t*>(db + o_ntk);
  w.chunk_off = reinterpret_cast<uint64_t*>(db + o_choff);
  w.page_off = reinterpret_cast<uint32_t*>(db + o_poff);
  w.blk_off = reinterpret_cast<uint32_t*>(db + o_boff);
  w.heads = reinterpret_cast<uint32_t*>(db + o_heads);
  w.chunk_span = reinterpret_cast<uint32_t*>(db + o_cspan);
  w.chunk_desc = with_desc ? reinterpret_cast<ChunkDesc*>(db + o_cdesc) : nullptr;
  w.chunk_shift = t.chunk_shift;
  // page allocation on the metadata stream (it overlaps the copy of the call before), the copy on the caller's
  k_alloc_scan<<<1, scan_threads(n), 0, p->meta>>>(p->view, w);
  k_alloc_fill<<<(unsigned)((std::max<uint64_t>(need, total_chunks) + 255) / 256), 256, 0, p->meta>>>(p->view, w, (uint32_t)need, total_chunks);
  p->gpu_launches += 2;
  if ((rc = meta_to(p, st)) != FT_OK) return rc;
  const bool f32 = src_dtype == FT_F32;
  mirror_write(p, n, slot, span_idx, n_tokens, t, f32);  // (the copy-engine path reads the page lists it leaves)
  if ((rc = launch_write_copies(p, w, total_chunks, f32, st, cx->counters, true, WriteArgs{n, slot, span_idx, n_tokens, src})) != FT_OK) return rc;
  if ((rc = ctx_release(p, cx, st)) != FT_OK) return rc;
  return end_producer(p, st);
}

extern "C" __attribute__((visibility("default"))) int32_t pool_free(ft_pool* p, const uint32_t* slot, uint32_t n, void* stream) {
  if (!p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (n == 0) return FT_OK;
  if (!slot) return FT_ERR_INVALID_ARG;
  const ft_pool_config& c = p->cfg;
  const uint32_t S = c.max_spans_per_sample;
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= c.max_samples) return FT_ERR_INVALID_ARG;
    ft_slot_mirror& sm = p->slots[slot[i]];
    if (sm.state == FT_SLOT_FREE || sm.named == p->call_seq) return FT_ERR_UNKNOWN_SAMPLE;  // free, or listed twice
    sm.named = p->call_seq;
  }
  uint64_t pages = 0, blocks = 0, text = 0, ns64 = 0;
  for (uint32_t i = 0; i < n; ++i) {
    const ft_slot_mirror& s = p->slots[slot[i]];
    for (uint32_t j = 0; j < s.n_spans; ++j) ns64 += p->spans[(uint64_t)slot[i] * S + j].written ? 1 : 0;
  }
  const uint32_t ns = (uint32_t)ns64;
  const size_t o_sid = 0, o_slot = (size_t)ns * 4;
  const size_t blob_bytes = align_up(o_slot + (size_t)n * 4, 256);
  const size_t o_poff = blob_bytes, o_boff = o_poff + (size_t)(ns + 1) * 4, o_toff = o_boff + (size_t)(ns + 1) * 4;
  const size_t o_tails = align_up(o_toff + (size_t)(n + 1) * 4, 16);
  const size_t total_bytes = o_tails + 16;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ft_call_ctx* cx = nullptr;
  int32_t rc = ctx_acquire(p, 0, blob_bytes, total_bytes, &cx);
  if (rc != FT_OK) return rc;
  uint8_t* hb = static_cast<uint8_t*>(cx->h);
  uint32_t* h_sid = reinterpret_cast<uint32_t*>(hb + o_sid);
  uint32_t k = 0;
  for (uint32_t i = 0; i < n; ++i) {
    const ft_slot_mirror& s = p->slots[slot[i]];
    for (uint32_t j = 0; j < s.n_spans; ++j) {
      const ft_span_mirror& m = p->spans[(uint64_t)slot[i] * S + j];
      if (!m.written) continue;
      h_sid[k++] = slot[i] * S + j;
      blocks += (m.npages + kListBlock - 1) / kListBlock;
      if (!s.remote) pages += m.npages;  // an imported sample's pages belong to the peer that wrote them
    }
    if (!s.remote) text += s.n_text_pages;
  }
  memcpy(hb + o_slot, slot, (size_t)n * 4);
  if ((rc = ctx_upload(p, cx, blob_bytes)) != FT_OK) return rc;
  uint8_t* db = static_cast<uint8_t*>(cx->d);
  FreeCall f;
  f.n_spans = ns; f.n_samples = n;
  f.span_id = reinterpret_cast<uint32_t*>(db + o_sid);
  f.slot = reinterpret_cast<uint32_t*>(db + o_slot);
  f.page_off = reinterpret_cast<uint32_t*>(db + o_poff);
  f.blk_off = reinterpret_cast<uint32_t*>(db + o_boff);
  f.tp_off = reinterpret_cast<uint32_t*>(db + o_toff);
  f.tails = reinterpret_cast<uint32_t*>(db + o_tails);
  // copies and assemblies still in flight (on the callers' streams) read these samples' tables and pages: the
  // metadata stream waits for the latest of each side, and for what the caller queued on `st` before this call
  if ((rc = meta_after_data(p)) != FT_OK) return rc;
  if ((rc = meta_after(p, st)) != FT_OK) return rc;
  k_free_scan<<<1, scan_threads(std::max(n, ns)), 0, p->meta>>>(p->view, f);
  const uint64_t items = pages + blocks + text;
  if (items) k_free_fill<<<(unsigned)((items + 255) / 256), 256, 0, p->meta>>>(p->view, f, (uint32_t)pages, (uint32_t)blocks, (uint32_t)text);
  k_free_clear<<<(std::max(n, ns) + 255) / 256, 256, 0, p->meta>>>(p->view, f);
  FT_CUDA(cudaGetLastError());
  if ((rc = ctx_release(p, cx, p->meta)) != FT_OK) return rc;
  p->gpu_launches += items ? 3 : 2;

  for (uint32_t i = 0; i < n; ++i) {
    ft_slot_mirror& s = p->slots[slot[i]];
    if (!s.remote)  // the pages go to the ring's tail as k_free_fill pushes them: spans by index, pages by ordinal
      for (uint32_t j = 0; j < s.n_spans; ++j)
      {
        const ft_span_mirror& m = p->spans[(uint64_t)slot[i] * S + j];
        uint32_t g = m.first_page;
        for (uint32_t k = 0; k < m.owned_pages; ++k) {
          p->h_ring[(p->h_ring_head + p->h_ring_count) % p->h_ring.size()] = g;
          ++p->h_ring_count;
          g = p->h_page_next[g];
        }
      }
    for (uint32_t j = 0; j < s.n_spans; ++j) p->spans[(uint64_t)slot[i] * S + j] = ft_span_mirror();
    p->live_samples--; p->live_spans -= s.n_spans;
    const uint64_t gen = s.generation + 1;
    s = ft_slot_mirror();
    s.generation = gen;
  }
  p->free_pages += pages; p->free_blocks += blocks; p->free_text_pages += text;
  p->free_epoch++;
  // what the caller queues on `st` next comes after the release
  if ((rc = meta_to(p, st)) != FT_OK) return rc;
  return end_producer(p, st);
}

extern "C" __attribute__((visibility("default"))) int32_t pool_ready_count(ft_pool* p, uint32_t* n_samples, uint64_t* n_tokens) {
  if (!p) return FT_ERR_INVALID_ARG;
  uint32_t n = 0;
  uint64_t tok = 0;
  for (const auto& e : p->ready_fifo) {
    const ft_slot_mirror& s = p->slots[e.first];
    if (s.state == FT_SLOT_READY && s.generation == e.second) { ++n; tok += s.seq_len; }
  }
  if (n_samples) *n_samples = n;
  if (n_tokens) *n_tokens = tok;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_take_ready(ft_pool* p, uint64_t min_tokens, uint32_t max_samples,
                                                                         uint32_t* slots_out, uint32_t* n_out, uint64_t* tokens_out) {
  if (!p || !n_out || (max_samples && !slots_out)) return FT_ERR_INVALID_ARG;
  *n_out = 0;
  if (tokens_out) *tokens_out = 0;
  // drop entries whose sample was freed (or freed and re-registered) since it became ready
  auto live = [&](const std::pair<uint32_t, uint64_t>& e) {
    const ft_slot_mirror& s = p->slots[e.first];
    return s.state == FT_SLOT_READY && s.generation == e.second;
  };
  uint64_t avail = 0;
  for (const auto& e : p->ready_fifo) if (live(e)) avail += p->slots[e.first].seq_len;
  if (avail < min_tokens || avail == 0) return FT_ERR_NOT_READY;  // not enough paired embeddings have accumulated
  uint32_t n = 0;
  uint64_t tok = 0;
  while (!p->ready_fifo.empty() && n < max_samples) {
    const auto e = p->ready_fifo.front();
    p->ready_fifo.pop_front();
    if (!live(e)) continue;
    slots_out[n++] = e.first;
    tok += p->slots[e.first].seq_len;
  }
  *n_out = n;
  if (tokens_out) *tokens_out = tok;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_status(ft_pool* p, int32_t* code, uint64_t* detail) {
  if (!p) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaDeviceSynchronize());
  unsigned long long key = 0;
  FT_CUDA(cudaMemcpy(&key, p->view.status, 8, cudaMemcpyDeviceToHost));
  p->status_base = p->call_seq;  // error keys count calls from here on
  if (key == ~0ull) { if (code) *code = 0; if (detail) *detail = 0; return FT_OK; }
  if (code) *code = -(int32_t)((key >> 32) & 0xF);
  if (detail) *detail = key & 0xFFFFFFFFull;
  FT_CUDA(cudaMemset(p->view.status, 0xFF, 8));
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_stats(ft_pool* p, ft_pool_stats* out) {
  if (!p || !out) return FT_ERR_INVALID_ARG;
  out->pages_total = p->cfg.hbm_pages + p->cfg.host_pages;
  out->pages_free = p->free_pages;
  out->hbm_pages = p->cfg.hbm_pages; out->host_pages = p->cfg.host_pages;
  out->text_pages_total = p->view.text_pages; out->text_pages_free = p->free_text_pages;
  out->live_samples = p->live_samples; out->live_spans = p->live_spans;
  out->bytes_written = p->bytes_written; out->bytes_gathered = p->bytes_gathered;
  out->gpu_launches = p->gpu_launches;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_get_tuning(ft_pool* p, ft_tuning* out) {
  if (!p || !out) return FT_ERR_INVALID_ARG;
  memset(out, 0, sizeof(*out));
  out->dev_ctas_per_sm = (uint32_t)p->dev_ctas_per_sm;
  out->scatter_ctas_per_sm = (uint32_t)(p->scatter_ctas_per_sm > 0 ? p->scatter_ctas_per_sm : 4);
  out->scatter_group = (uint32_t)(p->scatter_group > 0 ? p->scatter_group : 1);
  out->chunk_shift = (uint32_t)p->chunk_shift;
  out->host_ctas = (uint32_t)p->host_ctas; out->host_store_ctas = (uint32_t)p->host_store_ctas;
  out->gather_unroll = (uint32_t)p->gather_unroll;
  out->grad_ctas_per_sm = (uint32_t)p->grad_ctas_per_sm; out->grad_hot_threshold = (uint32_t)p->grad_hot_threshold;
  out->remote_ctas = (uint32_t)p->remote_ctas; out->peers_remote = (uint32_t)p->peers_remote;
  out->scatter_smem_carveout = (uint32_t)p->scatter_smem_carveout; out->gather_smem_carveout = (uint32_t)p->gather_smem_carveout;
  out->bulk_wait_limit_us = (uint32_t)(p->view.bulk_wait_ns / 1000); out->bulk_timeout_test = p->view.bulk_tx_slack ? 1u : 0u;
  out->host_copy_engine = (uint32_t)p->host_dma;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_set_tuning(ft_pool* p, const ft_tuning* in) {
  if (!p || !in) return FT_ERR_INVALID_ARG;
  const ft_tuning& t = *in;
  if (t.dev_ctas_per_sm > 8 || t.scatter_ctas_per_sm > 8 || t.grad_ctas_per_sm > 8) return FT_ERR_INVALID_ARG;
  if (t.chunk_shift && (t.chunk_shift < 14 || t.chunk_shift > 21)) return FT_ERR_INVALID_ARG;  // a warp's eighth holds a 2 KiB batch
  if (t.gather_unroll && t.gather_unroll != 4 && t.gather_unroll != 8) return FT_ERR_INVALID_ARG;
  if (t.host_ctas > 1024 || t.host_store_ctas > 1024 || t.remote_ctas > 1024 || t.scatter_group > (1u << 20) || t.peers_remote > 1 || t.scatter_smem_carveout > 100 || t.gather_smem_carveout > 100) return FT_ERR_INVALID_ARG;
  if (t.host_copy_engine > 1) return FT_ERR_INVALID_ARG;
  if (t.bulk_wait_limit_us && (t.bulk_wait_limit_us < 100 || t.bulk_wait_limit_us > 10000000)) return FT_ERR_INVALID_ARG;
  if (t.bulk_timeout_test > 1 || (t.bulk_timeout_test && (t.bulk_wait_limit_us == 0 || t.bulk_wait_limit_us > 100000))) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaDeviceSynchronize());  // no kernel of an earlier call is still being sized by the old values
  p->view.bulk_wait_ns = t.bulk_wait_limit_us ? (uint64_t)t.bulk_wait_limit_us * 1000 : kBulkWaitLimitNs;
  p->view.bulk_tx_slack = t.bulk_timeout_test ? 16u : 0u;
  p->host_dma = (int)t.host_copy_engine;
  p->dev_ctas_per_sm = (int)t.dev_ctas_per_sm;
  p->scatter_ctas_per_sm = (int)t.scatter_ctas_per_sm;
  p->scatter_group = (int)t.scatter_group;
  p->chunk_shift = (int)t.chunk_shift;
  p->host_ctas = t.host_ctas ? (int)t.host_ctas : 6;
  p->host_store_ctas = t.host_store_ctas ? (int)t.host_store_ctas : 8;
  p->gather_unroll = (int)t.gather_unroll;
  p->grad_ctas_per_sm = t.grad_ctas_per_sm ? (int)t.grad_ctas_per_sm : 6;
  p->grad_hot_threshold = (int)t.grad_hot_threshold;
  p->remote_ctas = t.remote_ctas ? (int)t.remote_ctas : 16;
  p->peers_remote = (int)t.peers_remote;
  {
    const int pct = t.scatter_smem_carveout ? (int)t.scatter_smem_carveout : 5;
    if (pct != p->scatter_smem_carveout) {
      const int32_t rc = scatter_set_carveout(pct);
      if (rc != FT_OK) return rc;
      p->scatter_smem_carveout = pct;
    }
    if ((int)t.gather_smem_carveout != p->gather_smem_carveout) {
      const int32_t rc = gather_set_carveout(t.gather_smem_carveout ? (int)t.gather_smem_carveout : (int)cudaSharedmemCarveoutDefault);
      if (rc != FT_OK) return rc;
      p->gather_smem_carveout = (int)t.gather_smem_carveout;
    }
  }
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_profile_enable(ft_pool* p, int32_t on) {
  if (!p) return FT_ERR_INVALID_ARG;
  p->profiling = on != 0;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_profile_read(ft_pool* p, ft_kernel_time* out) {
  if (!p || !out) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaDeviceSynchronize());
  for (int k = 0; k < FT_K_COUNT; ++k) { out[k].ms = 0; out[k].launches = 0; }
  for (auto& r : p->prof) {
    float ms = 0;
    if (cudaEventElapsedTime(&ms, r.e0, r.e1) == cudaSuccess) { out[r.kind].ms += ms; out[r.kind].launches++; }
    cudaEventDestroy(r.e0); cudaEventDestroy(r.e1);
  }
  p->prof.clear();
  cudaGetLastError();
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_debug_span_pages(ft_pool* p, uint32_t slot, uint32_t span, uint64_t* gva_out, uint32_t cap,
                                         uint32_t* n) {
  if (!p || slot >= p->cfg.max_samples) return FT_ERR_INVALID_ARG;
  const ft_slot_mirror& s = p->slots[slot];
  if (s.state == FT_SLOT_FREE) return FT_ERR_UNKNOWN_SAMPLE;
  if (span >= s.n_spans) return FT_ERR_INVALID_ARG;
  const uint32_t sid = slot * p->cfg.max_spans_per_sample + span;
  const uint32_t k = p->spans[sid].npages;
  if (n) *n = k;
  FT_CUDA(cudaDeviceSynchronize());
  const uint32_t want = std::min(k, cap);
  const uint32_t nb = (want + kListBlock - 1) / kListBlock;
  std::vector<uint32_t> blks(nb);
  if (nb) FT_CUDA(cudaMemcpy(blks.data(), p->view.sp_blocks + (uint64_t)sid * p->view.blocks_per_span, (size_t)nb * 4, cudaMemcpyDeviceToHost));
  for (uint32_t b = 0; b < nb; ++b) {
    const uint32_t cnt = std::min(kListBlock, want - b * kListBlock);
    FT_CUDA(cudaMemcpy(gva_out + (size_t)b * kListBlock, p->view.list_blocks + (uint64_t)blks[b] * kListBlock, (size_t)cnt * 8, cudaMemcpyDeviceToHost));
  }
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_debug_ring(ft_pool* p, uint32_t* out, uint64_t cap, uint64_t* n) {
  if (!p) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaDeviceSynchronize());
  RingState s;
  FT_CUDA(cudaMemcpy(&s, p->view.ring_state, sizeof(s), cudaMemcpyDeviceToHost));
  if (n) *n = s.count;
  std::vector<uint32_t> all(p->view.ring_cap);
  FT_CUDA(cudaMemcpy(all.data(), p->view.ring, (size_t)p->view.ring_cap * 4, cudaMemcpyDeviceToHost));
  for (uint64_t i = 0; i < s.count && i < cap; ++i) out[i] = all[(s.head + i) % p->view.ring_cap];
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_debug_translate(ft_pool* p, const uint64_t* gva, uint32_t n, uint32_t* kind, uint64_t* frame,
                                        uint64_t* offset, int32_t* status) {
  if (!p || (n && (!gva || !kind || !frame || !offset || !status))) return FT_ERR_INVALID_ARG;
  if (n == 0) return FT_OK;
  uint8_t* d = nullptr;
  const size_t W = p->cfg.world_size;
  const size_t bytes = (size_t)n * (8 + 4 + 8 + 8 + 4) + W * 24;
  FT_CUDA(cudaMalloc(&d, bytes));
  uint64_t* d_gva = reinterpret_cast<uint64_t*>(d);
  uint64_t* d_frame = d_gva + n;
  uint64_t* d_off = d_frame + n;
  uint64_t* d_bases = d_off + n;
  uint32_t* d_kind = reinterpret_cast<uint32_t*>(d_bases + 3 * W);
  int32_t* d_status = reinterpret_cast<int32_t*>(d_kind + n);
  std::vector<uint64_t> bases(3 * W, 0);
  for (size_t r = 0; r < W; ++r)
    if (r < p->peer_bases.size()) { bases[3 * r] = p->peer_bases[r][0]; bases[3 * r + 1] = p->peer_bases[r][1]; bases[3 * r + 2] = p->peer_bases[r][2]; }
  FT_CUDA(cudaMemcpy(d_bases, bases.data(), 24 * W, cudaMemcpyHostToDevice));
  FT_CUDA(cudaMemcpy(d_gva, gva, (size_t)n * 8, cudaMemcpyHostToDevice));
  k_debug_translate<<<(n + 255) / 256, 256>>>(p->view, d_gva, n, d_kind, d_frame, d_off, d_status, d_bases);
  p->gpu_launches++;
  FT_CUDA(cudaDeviceSynchronize());
  FT_CUDA(cudaMemcpy(kind, d_kind, (size_t)n * 4, cudaMemcpyDeviceToHost));
  FT_CUDA(cudaMemcpy(frame, d_frame, (size_t)n * 8, cudaMemcpyDeviceToHost));
  FT_CUDA(cudaMemcpy(offset, d_off, (size_t)n * 8, cudaMemcpyDeviceToHost));
  FT_CUDA(cudaMemcpy(status, d_status, (size_t)n * 4, cudaMemcpyDeviceToHost));
  FT_CUDA(cudaFree(d));
  return FT_OK;
}

// ------------------------------------------------------------------------------------------
// No-allocation variant of the producer write.  Its per-call scratch (descriptors in, scan outputs out) is a
// fixed array in the device image instead of the pool's growable cudaMalloc'd scratch, and the descriptors go
// up from a stack buffer instead of the pinned staging ring.  The kernels are the ones pool_write_embeddings
// launches.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[FT_NOALLOC_SCRATCH_BYTES];

namespace ft {
constexpr int kMaxDevices = 64;
// g_noalloc_scratch is a host-side stand-in here, not a device address: kernels get the address that
// cudaGetSymbolAddress returns for the device that is current (looked up once per device).
static void* g_noalloc_dev_ptr[kMaxDevices] = {};

static int32_t noalloc_scratch(int device, uint8_t** out) {
  if (device < 0 || device >= kMaxDevices) return FT_ERR_INVALID_ARG;
  if (!g_noalloc_dev_ptr[device]) {
    void* ptr = nullptr;
    FT_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    g_noalloc_dev_ptr[device] = ptr;
  }
  *out = static_cast<uint8_t*>(g_noalloc_dev_ptr[device]);
  return FT_OK;
}
}  // namespace ft

extern "C" __attribute__((visibility("default"))) int32_t pool_write_embeddings_noalloc(
    ft_pool* p, uint32_t n, const uint32_t* slot, const uint32_t* span_idx, const uint32_t* n_tokens,
    const void* const* src, uint32_t src_dtype, void* stream) {
  if (!p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (src_dtype != FT_BF16 && src_dtype != FT_F32) return FT_ERR_INVALID_ARG;
  if (n == 0) return FT_OK;
  if (n > FT_NOALLOC_MAX_SPANS) return FT_ERR_CAPACITY;  // call too large for the fixed scratch: split it
  if (!slot || !span_idx || !n_tokens || !src) return FT_ERR_INVALID_ARG;
  int cur = -1;
  FT_CUDA(cudaGetDevice(&cur));
  if (cur != p->device) return FT_ERR_INVALID_ARG;
  const uint32_t S = p->cfg.max_spans_per_sample;
  WriteTotals t;
  int32_t rc = check_write(p, n, slot, span_idx, n_tokens, src, &t, false);  // (no room for per-chunk records here)
  if (rc != FT_OK) return rc;

  // descriptor blob [src u64 n][span_id n][n_tokens n] in the host buffer pool_create made for this purpose
  const size_t o_src = 0, o_sid = (size_t)n * 8, o_ntk = o_sid + (size_t)n * 4;
  const size_t blob_bytes = align_up(o_ntk + (size_t)n * 4, 256);
  uint8_t* blob = p->noalloc_blob.data();
  for (uint32_t q = 0; q < n; ++q) {
    reinterpret_cast<uint64_t*>(blob + o_src)[q] = reinterpret_cast<uint64_t>(src[q]);
    reinterpret_cast<uint32_t*>(blob + o_sid)[q] = slot[q] * S + span_idx[q];
  }
  memcpy(blob + o_ntk, n_tokens, (size_t)n * 4);
  const size_t o_choff = blob_bytes, o_poff = align_up(o_choff + (size_t)(n + 1) * 8, 16);
  const size_t o_boff = o_poff + (size_t)(n + 1) * 4, o_heads = align_up(o_boff + (size_t)(n + 1) * 4, 16);
  constexpr size_t o_counters = FT_NOALLOC_SCRATCH_BYTES - 2 * sizeof(ClaimCounter);  // the array's last 32 bytes
  if (o_heads + 16 > o_counters) return FT_ERR_CAPACITY;
  uint8_t* db = nullptr;
  if ((rc = noalloc_scratch(p->device, &db)) != FT_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array still serves the previous no-allocation write of this pool until that call's copy has finished
  if (p->have_noalloc_ev) FT_CUDA(cudaStreamWaitEvent(p->meta, p->ev_noalloc, 0));
  // pageable source: cudaMemcpyAsync returns once the bytes have been taken, so the buffer is free again after it
  p->meta_seq++;
  FT_CUDA(cudaMemcpyAsync(db, blob, blob_bytes, cudaMemcpyHostToDevice, p->meta));
  WriteCall w;
  w.n = n;
  w.src = reinterpret_cast<uint64_t*>(db + o_src);
  w.span_id = reinterpret_cast<uint32_t*>(db + o_sid);
  w.n_tokens = reinterpret_cast<uint32_t*>(db + o_ntk);
  w.chunk_off = reinterpret_cast<uint64_t*>(db + o_choff);
  w.page_off = reinterpret_cast<uint32_t*>(db + o_poff);
  w.blk_off = reinterpret_cast<uint32_t*>(db + o_boff);
  w.heads = reinterpret_cast<uint32_t*>(db + o_heads);
  w.chunk_span = nullptr;  // the fixed scratch has no room for per-chunk tables: k_scatter searches chunk_off
  w.chunk_desc = nullptr;
  w.chunk_shift = t.chunk_shift;
  k_alloc_scan<<<1, scan_threads(n), 0, p->meta>>>(p->view, w);
  k_alloc_fill<<<(unsigned)((t.need + 255) / 256), 256, 0, p->meta>>>(p->view, w, (uint32_t)t.need, 0);
  p->gpu_launches += 2;
  if ((rc = meta_to(p, st)) != FT_OK) return rc;
  const bool f32 = src_dtype == FT_F32;
  // the claim counters of the copy kernels sit at the end of the array; they are zero whenever no kernel uses them
  mirror_write(p, n, slot, span_idx, n_tokens, t, f32);
  if ((rc = launch_write_copies(p, w, t.total_chunks, f32, st, reinterpret_cast<ClaimCounter*>(db + o_counters), true,
                                WriteArgs{n, slot, span_idx, n_tokens, src})) != FT_OK) return rc;
  FT_CUDA(cudaEventRecord(p->ev_noalloc, st));
  p->have_noalloc_ev = true;
  return end_producer(p, st);
}
