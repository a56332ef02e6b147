// More than one process in the GVA space (Sec. 3.2): every process exports its memory mapping, the others
// install it in their page tables, and from then on a GVA of any process's segment translates locally.
// Samples cross processes by descriptor only (lengths, spans, page GVAs): the consumer reads the bytes in place
// through the imported tables, with plain loads or bulk copies, never through the producer.
//
// Kernels in this file
//   k_export_lists   page GVAs and text-page GVAs of the exported samples into one contiguous buffer
//   k_import_pop     list blocks for the imported spans off the block ring
//   k_import_fill    sample / span tables and two-level page lists of the imported samples
#include <algorithm>
#include <cstring>

#include "flowpool_internal.cuh"

namespace ft {

constexpr uint64_t kMapMagic = 0x50414D4C4F4F5046ull;     // "FPOOLMAP"
constexpr uint64_t kSampleMagic = 0x504D534C4F4F5046ull;  // "FPOOLSMP"

struct MapHeader {
  uint64_t magic;
  uint64_t page_bytes, hbm_pages, host_pages, text_pages;
  uint64_t gva_hbm_start, gva_host_start, max_size;
  uint32_t rank, world_size;
};

struct SampleHeader {
  uint64_t magic;
  uint64_t total_pages, total_text_pages;
  uint32_t n, src_rank, total_spans, pad;
};
// then per sample {seq_len, n_spans, n_text_pages}, per span {pos, tokens, npages}, page GVAs, text-page GVAs

__device__ __forceinline__ uint32_t last_le_u32(const uint32_t* off, uint32_t n, uint32_t x) {
  uint32_t lo = 0, hi = n;
  while (hi - lo > 1) {
    uint32_t mid = (lo + hi) >> 1;
    if (off[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

struct ListCall {
  uint32_t n_spans, n_samples;
  const uint32_t* span_id;   // [n_spans] local span ids
  const uint32_t* page_off;  // [n_spans+1]
  const uint32_t* slot;      // [n_samples]
  const uint32_t* tp_off;    // [n_samples+1]
};

__global__ void k_export_lists(PoolView v, ListCall c, uint32_t total_pages, uint32_t total_text, uint64_t* out) {
  uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < total_pages) {
    const uint32_t q = last_le_u32(c.page_off, c.n_spans, t);
    out[t] = span_page_gva(v, c.span_id[q], t - c.page_off[q]);
    return;
  }
  t -= total_pages;
  if (t < total_text) {
    const uint32_t i = last_le_u32(c.tp_off, c.n_samples, t);
    out[total_pages + t] = v.s_text_pages[(uint64_t)c.slot[i] * v.text_pages_per_sample + (t - c.tp_off[i])];
  }
}

struct ImportCall {
  uint32_t n_spans, n_samples;
  const uint32_t *slot, *seq_len, *n_spans_of, *span_begin;  // per sample
  const uint32_t *span_pos, *span_tok, *span_npages;         // per span (concatenated)
  const uint32_t *page_off, *blk_off, *tp_off;               // prefix sums made on the host
  const uint64_t* gva;                                       // page GVAs then text-page GVAs
  uint32_t* head;                                            // [1] block ring head before the pops
  const uint4* span_grid;                                    // per span: token grid (T, H, W, 0), zero = none
};

__global__ void k_import_pop(PoolView v, ImportCall c, uint32_t total_blocks) {
  RingState s = *v.bring_state;
  c.head[0] = s.head;
  s.head = (uint32_t)(((uint64_t)s.head + total_blocks) % v.bring_cap);
  s.count -= total_blocks;
  *v.bring_state = s;
}

__global__ void __launch_bounds__(256) k_import_fill(PoolView v, ImportCall c, uint32_t total_pages, uint32_t total_text) {
  uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < c.n_samples) {  // tables
    const uint32_t slot = c.slot[t];
    v.s_seq_len[slot] = c.seq_len[t];
    v.s_n_spans[slot] = c.n_spans_of[t];
    v.s_flags[slot] = 1;  // imported
    for (uint32_t j = 0; j < c.n_spans_of[t]; ++j) {
      const uint32_t sid = slot * v.spans_per_sample + j, g = c.span_begin[t] + j;
      v.sp_pos[sid] = c.span_pos[g]; v.sp_tokens[sid] = c.span_tok[g]; v.sp_npages[sid] = c.span_npages[g];
      v.sp_grid[sid] = c.span_grid[g];
    }
  }
  if (t < total_pages) {
    const uint32_t q = last_le_u32(c.page_off, c.n_spans, t), o = t - c.page_off[q];
    // which sample does global span q belong to
    const uint32_t i = last_le_u32(c.span_begin, c.n_samples, q);
    const uint32_t sid = c.slot[i] * v.spans_per_sample + (q - c.span_begin[i]);
    const uint32_t blk = v.bring[(c.head[0] + c.blk_off[q] + o / kListBlock) % v.bring_cap];
    if (o % kListBlock == 0) v.sp_blocks[(uint64_t)sid * v.blocks_per_span + o / kListBlock] = blk;
    v.list_blocks[(uint64_t)blk * kListBlock + o % kListBlock] = c.gva[t];
    return;
  }
  t -= total_pages;
  if (t < total_text) {
    const uint32_t i = last_le_u32(c.tp_off, c.n_samples, t);
    v.s_text_pages[(uint64_t)c.slot[i] * v.text_pages_per_sample + (t - c.tp_off[i])] = c.gva[total_pages + t];
  }
}

}  // namespace ft

using namespace ft;

#define FT_API extern "C" __attribute__((visibility("default")))

FT_API int32_t pool_backing(ft_pool* p, void** hbm_base, void** host_base_device, void** text_base) {
  if (!p) return FT_ERR_INVALID_ARG;
  if (hbm_base) *hbm_base = p->hbm_base;
  if (host_base_device) *host_base_device = p->host_dev;
  if (text_base) *text_base = p->d_text;
  return FT_OK;
}

// Shareable handles of this pool's device slabs for a consumer in another process on the same node (Sec. 3.2:
// every process can address every other process's segment).  Only slabs the library allocated itself have a handle
// of their own; a caller-owned HBM slab is the caller's to share.
FT_API int32_t pool_ipc_export(ft_pool* p, ft_ipc_handles* out) {
  if (!p || !out) return FT_ERR_INVALID_ARG;
  static_assert(sizeof(cudaIpcMemHandle_t) == FT_IPC_HANDLE_BYTES, "handle size");
  memset(out, 0, sizeof(*out));
  if (p->cfg.hbm_pages) {
    if (!p->own_hbm) return FT_ERR_INVALID_ARG;
    cudaIpcMemHandle_t h;
    FT_CUDA(cudaIpcGetMemHandle(&h, p->hbm_base));
    memcpy(out->hbm, &h, sizeof(h));
    out->has_hbm = 1;
  }
  cudaIpcMemHandle_t t;
  FT_CUDA(cudaIpcGetMemHandle(&t, p->d_text));
  memcpy(out->text, &t, sizeof(t));
  out->has_text = 1;
  return FT_OK;
}

// Maps a peer process's slabs into this process: the base addresses pool_import_mapping wants.
FT_API int32_t pool_ipc_open(const ft_ipc_handles* in, void** hbm_base, void** text_base) {
  if (!in || !hbm_base || !text_base) return FT_ERR_INVALID_ARG;
  *hbm_base = nullptr; *text_base = nullptr;
  if (in->has_hbm) {
    cudaIpcMemHandle_t h;
    memcpy(&h, in->hbm, sizeof(h));
    FT_CUDA(cudaIpcOpenMemHandle(hbm_base, h, cudaIpcMemLazyEnablePeerAccess));
  }
  if (in->has_text) {
    cudaIpcMemHandle_t t;
    memcpy(&t, in->text, sizeof(t));
    const cudaError_t e = cudaIpcOpenMemHandle(text_base, t, cudaIpcMemLazyEnablePeerAccess);
    if (e != cudaSuccess) {
      if (*hbm_base) { cudaIpcCloseMemHandle(*hbm_base); *hbm_base = nullptr; }
      return cuda_fail(e, "cudaIpcOpenMemHandle(text)");
    }
  }
  return FT_OK;
}

FT_API int32_t pool_ipc_close(void* hbm_base, void* text_base) {
  if (hbm_base) FT_CUDA(cudaIpcCloseMemHandle(hbm_base));
  if (text_base) FT_CUDA(cudaIpcCloseMemHandle(text_base));
  return FT_OK;
}

FT_API int32_t pool_export_mapping(ft_pool* p, void* buf, uint64_t cap, uint64_t* bytes) {
  if (!p) return FT_ERR_INVALID_ARG;
  const uint64_t need = sizeof(MapHeader) + 4 * (p->cfg.hbm_pages + p->cfg.host_pages);
  if (bytes) *bytes = need;
  if (!buf) return FT_OK;  // size query
  if (cap < need) return FT_ERR_CAPACITY;
  MapHeader h{};
  h.magic = kMapMagic;
  h.page_bytes = p->cfg.page_bytes; h.hbm_pages = p->cfg.hbm_pages; h.host_pages = p->cfg.host_pages;
  h.text_pages = p->view.text_pages;
  h.gva_hbm_start = p->cfg.gva_hbm_start; h.gva_host_start = p->cfg.gva_host_start; h.max_size = p->cfg.max_size;
  h.rank = p->cfg.rank; h.world_size = p->cfg.world_size;
  uint8_t* b = static_cast<uint8_t*>(buf);
  memcpy(b, &h, sizeof(h));
  if (p->cfg.hbm_pages) memcpy(b + sizeof(h), p->bind_hbm.data(), 4 * p->cfg.hbm_pages);
  if (p->cfg.host_pages) memcpy(b + sizeof(h) + 4 * p->cfg.hbm_pages, p->bind_host.data(), 4 * p->cfg.host_pages);
  return FT_OK;
}

FT_API int32_t pool_import_mapping(ft_pool* p, const void* buf, uint64_t bytes, void* peer_hbm_base, void* peer_host_base,
                                   void* peer_text_base) {
  if (!p || !buf || bytes < sizeof(MapHeader)) return FT_ERR_INVALID_ARG;
  MapHeader h;
  memcpy(&h, buf, sizeof(h));
  const ft_pool_config& c = p->cfg;
  if (h.magic != kMapMagic || bytes != sizeof(MapHeader) + 4 * (h.hbm_pages + h.host_pages)) return FT_ERR_INVALID_ARG;
  if (h.world_size != c.world_size || h.rank >= c.world_size || h.rank == c.rank) return FT_ERR_INVALID_ARG;
  if (h.page_bytes != c.page_bytes || h.gva_hbm_start != c.gva_hbm_start || h.gva_host_start != c.gva_host_start ||
      h.max_size != c.max_size)
    return FT_ERR_INVALID_ARG;  // not the same GVA space
  if (p->peer_imported[h.rank]) return FT_ERR_SLOT_IN_USE;
  if ((h.hbm_pages && !peer_hbm_base) || (h.host_pages && !peer_host_base) || (h.text_pages && !peer_text_base)) return FT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(peer_hbm_base) | reinterpret_cast<uintptr_t>(peer_host_base) | reinterpret_cast<uintptr_t>(peer_text_base)) & 255)
    return FT_ERR_INVALID_ARG;
  const uint8_t* b = static_cast<const uint8_t*>(buf) + sizeof(MapHeader);
  const uint64_t entries = h.hbm_pages + h.host_pages + h.text_pages;
  uint64_t* d_pte = nullptr;
  uint32_t* d_bind = nullptr;
  FT_CUDA(cudaMalloc(&d_pte, std::max<uint64_t>(entries, 1) * 8));
  cudaError_t e = cudaMalloc(&d_bind, std::max<uint64_t>(h.hbm_pages + h.host_pages, 1) * 4);
  if (e != cudaSuccess) { cudaFree(d_pte); return ft::cuda_fail(e, "cudaMalloc(peer bind)"); }
  auto fail = [&](cudaError_t err, const char* what) { cudaFree(d_pte); cudaFree(d_bind); return ft::cuda_fail(err, what); };
  if (h.hbm_pages + h.host_pages) {
    e = cudaMemcpy(d_bind, b, 4 * (h.hbm_pages + h.host_pages), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) return fail(e, "cudaMemcpy(peer bind)");
  }
  auto blocks = [](uint64_t n) { return (unsigned)((n + 255) / 256); };
  uint64_t* pte_hbm = d_pte;
  uint64_t* pte_host = d_pte + h.hbm_pages;
  uint64_t* pte_text = pte_host + h.host_pages;
  // where the peer's HBM slab lives: frames of another device are remote (read over NVLink by a launch of their own)
  bool remote = p->peers_remote != 0;
  if (h.hbm_pages && !remote) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, peer_hbm_base) == cudaSuccess && at.type == cudaMemoryTypeDevice && at.device != p->device) remote = true;
    cudaGetLastError();
  }
  if (h.hbm_pages) k_page_table_init<<<blocks(h.hbm_pages), 256>>>(pte_hbm, d_bind, h.hbm_pages, reinterpret_cast<uint64_t>(peer_hbm_base), h.page_bytes, kPteValid | (remote ? kPteRemote : 0));
  if (h.host_pages) k_page_table_init<<<blocks(h.host_pages), 256>>>(pte_host, d_bind + h.hbm_pages, h.host_pages, reinterpret_cast<uint64_t>(peer_host_base), h.page_bytes, kPteValid | kPteHost);
  if (h.text_pages) k_page_table_init<<<blocks(h.text_pages), 256>>>(pte_text, nullptr, h.text_pages, reinterpret_cast<uint64_t>(peer_text_base), FT_TEXT_PAGE_BYTES, kPteValid | kPteText);
  p->gpu_launches += 3;
  PeerTables pt{pte_hbm, pte_host, pte_text, h.hbm_pages, h.host_pages, h.text_pages};
  e = cudaMemcpy(const_cast<PeerTables*>(p->view.peers) + h.rank, &pt, sizeof(pt), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return fail(e, "cudaMemcpy(peer tables)");
  e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return fail(e, "cudaDeviceSynchronize(import mapping)");
  cudaFree(d_bind);
  p->peer_allocs.push_back(d_pte);
  p->peer_imported[h.rank] = 1;
  if (h.host_pages) p->peer_host_frames = true;
  if (h.hbm_pages && remote) p->peer_remote_frames = true;
  p->peer_bases[h.rank] = {reinterpret_cast<uint64_t>(peer_hbm_base), reinterpret_cast<uint64_t>(peer_host_base), reinterpret_cast<uint64_t>(peer_text_base)};
  return FT_OK;
}

FT_API int32_t pool_export_samples(ft_pool* p, const uint32_t* slot, uint32_t n, void* buf, uint64_t cap, uint64_t* bytes,
                                   void* stream) {
  if (!p || (n && !slot)) return FT_ERR_INVALID_ARG;
  const ft_pool_config& c = p->cfg;
  const uint32_t S = c.max_spans_per_sample;
  uint64_t total_pages = 0, total_text = 0, total_spans = 0;
  std::vector<uint8_t> seen(c.max_samples, 0);
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= c.max_samples) return FT_ERR_INVALID_ARG;
    const ft_slot_mirror& s = p->slots[slot[i]];
    if (s.state == FT_SLOT_FREE) return FT_ERR_UNKNOWN_SAMPLE;
    if (seen[slot[i]]) return FT_ERR_INVALID_ARG;
    seen[slot[i]] = 1;
    if (s.state != FT_SLOT_READY) return FT_ERR_NOT_READY;  // only paired samples leave their process
    for (uint32_t j = 0; j < s.n_spans; ++j) total_pages += p->spans[(uint64_t)slot[i] * S + j].npages;
    total_spans += s.n_spans;
    total_text += s.n_text_pages;
  }
  const uint64_t need = sizeof(SampleHeader) + 12ull * n + 24ull * total_spans + 8ull * (total_pages + total_text);
  if (bytes) *bytes = need;
  if (!buf) return FT_OK;  // size query
  if (cap < need) return FT_ERR_CAPACITY;
  if (total_pages + total_text > 0xFFFFFFFFull) return FT_ERR_INVALID_ARG;
  uint8_t* out = static_cast<uint8_t*>(buf);
  SampleHeader h{};
  h.magic = kSampleMagic; h.total_pages = total_pages; h.total_text_pages = total_text;
  h.n = n; h.src_rank = c.rank; h.total_spans = (uint32_t)total_spans;
  memcpy(out, &h, sizeof(h));
  uint32_t* ps = reinterpret_cast<uint32_t*>(out + sizeof(h));
  uint32_t* pp = ps + 3ull * n;
  uint64_t* pg = reinterpret_cast<uint64_t*>(pp + 6ull * total_spans);
  // descriptors for the list kernel
  std::vector<uint32_t> span_id, page_off(1, 0), tp_off(1, 0);
  for (uint32_t i = 0; i < n; ++i) {
    const ft_slot_mirror& s = p->slots[slot[i]];
    ps[3 * i] = s.seq_len; ps[3 * i + 1] = s.n_spans; ps[3 * i + 2] = s.n_text_pages;
    for (uint32_t j = 0; j < s.n_spans; ++j) {
      const ft_span_mirror& m = p->spans[(uint64_t)slot[i] * S + j];
      *pp++ = m.pos; *pp++ = m.tokens; *pp++ = m.npages;
      *pp++ = m.grid[0]; *pp++ = m.grid[1]; *pp++ = m.grid[2];  // the span's token grid travels with it
      span_id.push_back(slot[i] * S + j);
      page_off.push_back(page_off.back() + m.npages);
    }
    tp_off.push_back(tp_off.back() + s.n_text_pages);
  }
  if (n == 0 || total_pages + total_text == 0) return FT_OK;
  const uint32_t ns = (uint32_t)span_id.size();
  const size_t o_sid = 0, o_poff = (size_t)ns * 4, o_slot = o_poff + (size_t)(ns + 1) * 4, o_tpoff = o_slot + (size_t)n * 4;
  const size_t blob_bytes = align_up_sz(o_tpoff + (size_t)(n + 1) * 4, 256);
  const size_t o_out = blob_bytes, total_bytes = o_out + 8 * (total_pages + total_text);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ft_call_ctx* cx = nullptr;
  int32_t rc = ctx_acquire(p, 1, blob_bytes, total_bytes, &cx);
  if (rc != FT_OK) return rc;
  uint8_t* hb = static_cast<uint8_t*>(cx->h);
  if (ns) memcpy(hb + o_sid, span_id.data(), (size_t)ns * 4);
  memcpy(hb + o_poff, page_off.data(), (size_t)(ns + 1) * 4);
  memcpy(hb + o_slot, slot, (size_t)n * 4);
  memcpy(hb + o_tpoff, tp_off.data(), (size_t)(n + 1) * 4);
  if ((rc = ctx_upload(p, cx, blob_bytes)) != FT_OK) return rc;
  uint8_t* db = static_cast<uint8_t*>(cx->d);
  ListCall lc{ns, n, reinterpret_cast<uint32_t*>(db + o_sid), reinterpret_cast<uint32_t*>(db + o_poff),
              reinterpret_cast<uint32_t*>(db + o_slot), reinterpret_cast<uint32_t*>(db + o_tpoff)};
  const uint64_t items = total_pages + total_text;
  // the page lists are metadata: the list kernel runs on the metadata stream, behind the allocations that wrote them
  k_export_lists<<<(unsigned)((items + 255) / 256), 256, 0, p->meta>>>(p->view, lc, (uint32_t)total_pages, (uint32_t)total_text,
                                                                       reinterpret_cast<uint64_t*>(db + o_out));
  p->gpu_launches++;
  FT_CUDA(cudaMemcpyAsync(pg, db + o_out, 8 * items, cudaMemcpyDeviceToHost, p->meta));
  if ((rc = ctx_release(p, cx, p->meta)) != FT_OK) return rc;
  FT_CUDA(cudaStreamSynchronize(p->meta));
  // a consumer will read the pages themselves as soon as it holds the descriptors: the copies that fill them (on
  // the producer side's stream and on `stream`) are complete when this call returns
  if (p->have_producer_ev) FT_CUDA(cudaEventSynchronize(p->ev_producer));
  FT_CUDA(cudaStreamSynchronize(st));
  return FT_OK;
}

FT_API int32_t pool_import_samples(ft_pool* p, const uint32_t* local_slot, uint32_t n, const void* buf, uint64_t bytes,
                                   void* stream) {
  if (!p || !buf || bytes < sizeof(SampleHeader) || (n && !local_slot)) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  SampleHeader h;
  memcpy(&h, buf, sizeof(h));
  if (h.magic != kSampleMagic || h.n != n) return FT_ERR_INVALID_ARG;
  if (bytes != sizeof(SampleHeader) + 12ull * n + 24ull * h.total_spans + 8ull * (h.total_pages + h.total_text_pages)) return FT_ERR_INVALID_ARG;
  const ft_pool_config& c = p->cfg;
  if (h.src_rank >= c.world_size || !p->peer_imported[h.src_rank]) return FT_ERR_INVALID_ARG;  // mapping first
  if (n == 0) return FT_OK;
  const uint8_t* in = static_cast<const uint8_t*>(buf);
  const uint32_t* ps = reinterpret_cast<const uint32_t*>(in + sizeof(h));
  const uint32_t* pp = ps + 3ull * n;
  const uint64_t* pg = reinterpret_cast<const uint64_t*>(pp + 6ull * h.total_spans);
  const uint32_t S = c.max_spans_per_sample, TPS = p->view.text_pages_per_sample, MB = p->view.blocks_per_span;
  std::vector<uint8_t> seen(c.max_samples, 0);
  uint64_t spans = 0, pages = 0, text = 0, blocks = 0;
  for (uint32_t i = 0; i < n; ++i) {
    if (local_slot[i] >= c.max_samples) return FT_ERR_INVALID_ARG;
    if (p->slots[local_slot[i]].state != FT_SLOT_FREE || seen[local_slot[i]]) return FT_ERR_SLOT_IN_USE;
    seen[local_slot[i]] = 1;
    const uint32_t seq_len = ps[3 * i], nsp = ps[3 * i + 1], ntp = ps[3 * i + 2];
    if (seq_len == 0 || ntp != (seq_len + kTextPageIds - 1) / kTextPageIds) return FT_ERR_INVALID_ARG;
    if (seq_len > c.max_seq_len || nsp > S || ntp > TPS) return FT_ERR_CAPACITY;
    if (spans + nsp > h.total_spans) return FT_ERR_INVALID_ARG;
    for (uint32_t j = 0; j < nsp; ++j) {
      const uint32_t* rec = pp + 6 * (spans + j);
      const uint32_t np = rec[2];
      if ((np + kListBlock - 1) / kListBlock > MB) return FT_ERR_CAPACITY;
      if (rec[3] | rec[4] | rec[5]) {  // a token grid: extents whose product is the token count
        const uint64_t tokens = rec[1], th = (uint64_t)rec[3] * rec[4];
        if (!rec[3] || !rec[4] || !rec[5] || th > tokens || th * rec[5] != tokens) return FT_ERR_INVALID_ARG;
      }
      pages += np; blocks += (np + kListBlock - 1) / kListBlock;
    }
    spans += nsp; text += ntp;
  }
  if (spans != h.total_spans || pages != h.total_pages || text != h.total_text_pages) return FT_ERR_INVALID_ARG;
  if (blocks > p->free_blocks) return FT_ERR_CAPACITY;
  if (pages + text > 0xFFFFFFFFull) return FT_ERR_INVALID_ARG;

  // upload: per-sample arrays, per-span arrays, prefix sums, GVAs
  const uint32_t ns = (uint32_t)spans;
  std::vector<uint32_t> seq(n), nsp(n), sbeg(n + 1, 0), pos(ns), tok(ns), npg(ns), poff(ns + 1, 0), boff(ns + 1, 0), tpoff(n + 1, 0);
  std::vector<uint4> grid(ns);
  for (uint32_t i = 0, g = 0; i < n; ++i) {
    seq[i] = ps[3 * i]; nsp[i] = ps[3 * i + 1];
    sbeg[i + 1] = sbeg[i] + nsp[i];
    tpoff[i + 1] = tpoff[i] + ps[3 * i + 2];
    for (uint32_t j = 0; j < nsp[i]; ++j, ++g) {
      pos[g] = pp[6 * g]; tok[g] = pp[6 * g + 1]; npg[g] = pp[6 * g + 2];
      grid[g] = make_uint4(pp[6 * g + 3], pp[6 * g + 4], pp[6 * g + 5], 0);
      poff[g + 1] = poff[g] + npg[g];
      boff[g + 1] = boff[g] + (npg[g] + kListBlock - 1) / kListBlock;
    }
  }
  size_t off = 0;
  auto take = [&](size_t b) { size_t o = off; off = align_up_sz(off + b, 16); return o; };
  const size_t o_gva = take(8 * (pages + text));
  const size_t o_slot = take(4ull * n), o_seq = take(4ull * n), o_nsp = take(4ull * n), o_sbeg = take(4ull * (n + 1));
  const size_t o_pos = take(4ull * ns), o_tok = take(4ull * ns), o_npg = take(4ull * ns);
  const size_t o_poff = take(4ull * (ns + 1)), o_boff = take(4ull * (ns + 1)), o_tpoff = take(4ull * (n + 1));
  const size_t o_grid = take(16ull * ns);
  const size_t blob_bytes = align_up_sz(off, 256), o_head = blob_bytes, total_bytes = o_head + 16;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ft_call_ctx* cx = nullptr;
  int32_t rc = ctx_acquire(p, 0, blob_bytes, total_bytes, &cx);
  if (rc != FT_OK) return rc;
  uint8_t* hb = static_cast<uint8_t*>(cx->h);
  memcpy(hb + o_gva, pg, 8 * (pages + text));
  memcpy(hb + o_slot, local_slot, 4ull * n);
  memcpy(hb + o_seq, seq.data(), 4ull * n);
  memcpy(hb + o_nsp, nsp.data(), 4ull * n);
  memcpy(hb + o_sbeg, sbeg.data(), 4ull * (n + 1));
  if (ns) memcpy(hb + o_grid, grid.data(), 16ull * ns);
  if (ns) { memcpy(hb + o_pos, pos.data(), 4ull * ns); memcpy(hb + o_tok, tok.data(), 4ull * ns); memcpy(hb + o_npg, npg.data(), 4ull * ns); }
  memcpy(hb + o_poff, poff.data(), 4ull * (ns + 1));
  memcpy(hb + o_boff, boff.data(), 4ull * (ns + 1));
  memcpy(hb + o_tpoff, tpoff.data(), 4ull * (n + 1));
  if ((rc = ctx_upload(p, cx, blob_bytes)) != FT_OK) return rc;
  uint8_t* db = static_cast<uint8_t*>(cx->d);
  auto U = [&](size_t o) { return reinterpret_cast<uint32_t*>(db + o); };
  ImportCall ic{ns, n, U(o_slot), U(o_seq), U(o_nsp), U(o_sbeg), U(o_pos), U(o_tok), U(o_npg), U(o_poff), U(o_boff), U(o_tpoff),
                reinterpret_cast<uint64_t*>(db + o_gva), U(o_head), reinterpret_cast<const uint4*>(db + o_grid)};
  k_import_pop<<<1, 1, 0, p->meta>>>(p->view, ic, (uint32_t)blocks);
  const uint64_t items = std::max<uint64_t>(pages + text, n);
  k_import_fill<<<(unsigned)((items + 255) / 256), 256, 0, p->meta>>>(p->view, ic, (uint32_t)pages, (uint32_t)text);
  FT_CUDA(cudaGetLastError());
  if ((rc = ctx_release(p, cx, p->meta)) != FT_OK) return rc;
  p->gpu_launches += 2;

  for (uint32_t i = 0, g = 0; i < n; ++i) {
    ft_slot_mirror& s = p->slots[local_slot[i]];
    s.state = FT_SLOT_READY; s.remote = true;
    ready_push(p, local_slot[i]);
    s.seq_len = seq[i]; s.n_spans = nsp[i]; s.spans_written = nsp[i]; s.n_text_pages = ps[3 * i + 2];
    for (uint32_t j = 0; j < nsp[i]; ++j, ++g) {
      ft_span_mirror& m = p->spans[(uint64_t)local_slot[i] * S + j];
      m.pos = pos[g]; m.tokens = tok[g]; m.npages = npg[g]; m.written = true;
      m.grid[0] = grid[g].x; m.grid[1] = grid[g].y; m.grid[2] = grid[g].z;
    }
    p->live_samples++; p->live_spans += nsp[i];
  }
  p->free_blocks -= blocks;
  if ((rc = meta_to(p, st)) != FT_OK) return rc;  // what the caller queues on `stream` next sees the imported samples
  return end_producer(p, st);
}
