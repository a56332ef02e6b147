// Internal declarations of the flowpool CUDA library (sm_100a).  Not part of the ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <array>
#include <deque>
#include <utility>
#include <vector>

#include "../../include/flowpool.h"

namespace ft {

constexpr uint32_t kTextPageIds = 1024;       // ids per 4 KiB text page
constexpr uint32_t kListBlock = 64;           // page GVAs per list block (two-level span page lists)
constexpr uint32_t kNone = 0xFFFFFFFFu;
constexpr uint64_t kPteValid = 1, kPteHost = 2, kPteText = 4, kPteRemote = 8, kPteFlagMask = 0xFF;  // Remote: HBM of another GPU

struct RingState {
  uint32_t head;   // index of the oldest free entry
  uint32_t count;  // free entries
};

// Page tables of one process of the GVA space, as this process holds them (Sec. 3.2: every process keeps the
// collected page tables locally).  Entry 'rank' is this process's own binding; the others are filled by
// pool_import_mapping and stay empty (no pages) until then.
struct PeerTables {
  const uint64_t* pte_hbm;
  const uint64_t* pte_host;
  const uint64_t* pte_text;
  uint64_t hbm_pages, host_pages, text_pages;
};

// Everything a kernel needs to know about a pool; passed by value.
struct PoolView {
  // GVA layout (Sec. 3.2): two regions, per-process segments
  uint64_t region_start[2];  // start_HBM, start_DRAM
  uint64_t region_bytes;     // world_size * max_size
  uint64_t max_size;
  uint64_t seg_base[2];      // this process's segment bases
  uint64_t text_gva_base;    // first text page: seg_base[0] + hbm_pages * page_bytes
  uint32_t rank, page_shift;
  uint64_t page_bytes, hbm_pages, host_pages, text_pages;
  uint32_t hidden, row_bytes;
  int32_t placeholder_id;
  uint32_t max_samples, spans_per_sample, text_pages_per_sample, blocks_per_span;
  // page tables: entry = device-visible frame address | flags
  const uint64_t* pte_hbm;
  const uint64_t* pte_host;
  const uint64_t* pte_text;
  const PeerTables* peers;   // [world_size] device array: every process's tables (own entry included)
  uint32_t world_size;
  // FIFO free rings
  uint32_t* ring;   RingState* ring_state;   uint32_t ring_cap;    // embedding pages (global page index)
  uint32_t* tring;  RingState* tring_state;  uint32_t tring_cap;   // text pages
  uint32_t* bring;  RingState* bring_state;  uint32_t bring_cap;   // list blocks
  // sample table (by slot)
  uint32_t* s_seq_len;
  uint32_t* s_n_spans;
  uint64_t* s_text_pages;  // [max_samples][text_pages_per_sample] text page GVA (own or a peer's)
  uint32_t* s_flags;       // bit 0: the sample was imported (its pages and text pages belong to a peer)
  // span table (span id = slot * spans_per_sample + j)
  uint32_t* sp_pos;
  uint32_t* sp_tokens;
  uint32_t* sp_npages;     // 0 until written
  uint32_t* sp_blocks;     // [span id][blocks_per_span] list block index
  uint64_t* list_blocks;   // [bring_cap][kListBlock] page GVAs
  uint4* sp_grid;          // token grid (T, H, W, 0) of a span; all zero = none given
  unsigned long long* status;  // first asynchronous error key; ~0 = none
  // the bulk-copy rings' bounded waits: limit per wait, and bytes a staged load announces beyond what it requests
  // (0 in use; 16 only under the timeout test, whose loads are therefore never seen complete)
  uint64_t bulk_wait_ns;
  uint32_t bulk_tx_slack;
};

// key = seq << 36 | (-code) << 32 | detail ; the smallest key is reported.  seq = calls since the status word was
// last read (28 bits: pool_status restarts the count), so the order of the keys is the order of the calls.
constexpr uint64_t kStatusSeqMask = (1ull << 28) - 1;
__device__ __forceinline__ void note_error(const PoolView& v, uint64_t seq, int32_t code, uint32_t detail) {
  unsigned long long key = ((seq & kStatusSeqMask) << 36) | ((unsigned long long)((uint32_t)(-code) & 15u) << 32) | detail;
  atomicMin(v.status, key);
}

// Work counters of the persistent data kernels.  A kernel claims its work units in order with atomicAdd(claim) and,
// when a CTA runs out of work, reports with atomicAdd(done): the last CTA of the grid puts both words back to zero,
// so a counter pair is zero whenever no kernel is using it and no launch needs a memset in front of it.
struct ClaimCounter {
  unsigned long long claim, done;
};
__device__ __forceinline__ void claim_release(ClaimCounter* c) {  // one thread per CTA, after its last claim
  __threadfence();
  if (atomicAdd(&c->done, 1ull) == (unsigned long long)gridDim.x * gridDim.y - 1) {
    c->claim = 0; c->done = 0;
    __threadfence();
  }
}

__device__ __forceinline__ uint64_t page_gva(const PoolView& v, uint32_t global_page) {
  return global_page < v.hbm_pages ? v.seg_base[0] + (uint64_t)global_page * v.page_bytes
                                   : v.seg_base[1] + ((uint64_t)global_page - v.hbm_pages) * v.page_bytes;
}

// inverse of page_gva for a page GVA produced by it
__device__ __forceinline__ uint32_t global_page_of(const PoolView& v, uint64_t gva) {
  uint64_t d = gva - v.seg_base[1];
  if (d < v.max_size) return (uint32_t)(v.hbm_pages + (d >> v.page_shift));
  return (uint32_t)((gva - v.seg_base[0]) >> v.page_shift);
}

// GVA -> page-table entry (+ byte offset inside the frame).  Purely local: region by
// interval test, process by division, virtual page number by shift (Sec. 3.2).
// Returns 0 (no valid bit) when the GVA does not translate.
__device__ __forceinline__ uint64_t translate(const PoolView& v, uint64_t gva, uint64_t* offset) {
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    uint64_t d = gva - v.region_start[t];
    if (d >= v.region_bytes) continue;
    const uint64_t proc = d / v.max_size, o = d - proc * v.max_size;
    uint64_t hbm_pages = v.hbm_pages, host_pages = v.host_pages, text_pages = v.text_pages;
    const uint64_t *pte_hbm = v.pte_hbm, *pte_host = v.pte_host, *pte_text = v.pte_text;
    if (proc != v.rank) {  // another process's segment: its imported tables (no pages if never imported)
      const PeerTables pt = v.peers[proc];
      hbm_pages = pt.hbm_pages; host_pages = pt.host_pages; text_pages = pt.text_pages;
      pte_hbm = pt.pte_hbm; pte_host = pt.pte_host; pte_text = pt.pte_text;
    }
    const uint64_t pages = t == 0 ? hbm_pages : host_pages;
    const uint64_t vpn = o >> v.page_shift;
    if (vpn < pages) {
      *offset = o & (v.page_bytes - 1);
      return t == 0 ? pte_hbm[vpn] : pte_host[vpn];
    }
    if (t == 0) {
      const uint64_t ot = o - (pages << v.page_shift);
      const uint64_t tp = ot / FT_TEXT_PAGE_BYTES;
      if (tp < text_pages) {
        *offset = ot % FT_TEXT_PAGE_BYTES;
        return pte_text[tp];
      }
    }
    return 0;
  }
  return 0;
}

// page GVA of ordinal o of a span, through the two-level list
__device__ __forceinline__ uint64_t span_page_gva(const PoolView& v, uint32_t span_id, uint32_t o) {
  uint32_t blk = v.sp_blocks[(uint64_t)span_id * v.blocks_per_span + o / kListBlock];
  return v.list_blocks[(uint64_t)blk * kListBlock + o % kListBlock];
}

// block-wide exclusive scan of one value per thread (blockDim.x a multiple of 32, <= 1024);
// returns the exclusive prefix, *total = block sum.  All threads must call.
__device__ __forceinline__ uint64_t block_exclusive_scan(uint64_t x, uint64_t* total) {
  __shared__ uint64_t warp_sums[32];
  __shared__ uint64_t block_total;
  const unsigned lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  uint64_t incl = x;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    uint64_t y = __shfl_up_sync(0xFFFFFFFFu, incl, d);
    if (lane >= (unsigned)d) incl += y;
  }
  __syncthreads();  // protect warp_sums from a previous call
  if (lane == 31) warp_sums[wid] = incl;
  __syncthreads();
  if (wid == 0) {
    uint64_t s = lane < nw ? warp_sums[lane] : 0, si = s;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      uint64_t y = __shfl_up_sync(0xFFFFFFFFu, si, d);
      if (lane >= (unsigned)d) si += y;
    }
    if (lane < nw) warp_sums[lane] = si - s;
    if (lane == 31) block_total = si;
  }
  __syncthreads();
  *total = block_total;
  return warp_sums[wid] + incl - x;
}

// ---- plan: device arrays and host summary -------------------------------------------------
struct PlanView {
  uint32_t n, n_mb, n_ranks;
  const uint32_t* mb_samples;        // [n] slots, plan order
  const uint32_t* plan_sample_mb;    // [n] microbatch of the sample at plan position q
  const uint64_t* sample_row_off;    // [n+1] first output row of the sample at plan position q
  const uint32_t* mb_sample_off;     // [n_mb+1]
  const uint64_t* mb_row_off;        // [n_mb+1]
  const uint32_t* tile_first_sample; // [ceil(rows/32)] plan position of the sample holding row 32*T
  const uint64_t* row_src;           // [rows] row words (kind | position | token id or span id), or nullptr
};

}  // namespace ft

// ---- host-side objects -------------------------------------------------------------------
struct ft_plan {
  ft_pool* pool;
  ft_plan_config cfg;
  uint32_t n = 0, n_mb = 0;
  uint64_t total_tokens = 0;
  uint32_t max_mb_tokens = 0;
  uint64_t free_epoch = 0;
  std::vector<uint32_t> slots;            // caller's order
  std::vector<uint64_t> slot_generation;
  std::vector<uint32_t> h_mb_sample_off;  // host copies used to size gathers
  std::vector<uint64_t> h_mb_row_off;
  void* d_block = nullptr;                // one device block holding every array below (from the pool's block cache)
  size_t block_cap = 0;
  cudaStream_t last_stream = nullptr;     // stream of the plan's latest device work (creation, then gathers)
  uint32_t *d_slots, *d_len, *d_sample_mb, *d_sample_rank, *d_mb_sample_off, *d_mb_samples, *d_plan_sample_mb;
  uint32_t *d_mb_tokens, *d_mb_lmax, *d_mb_residual, *d_mb_count, *d_mb_bucket, *d_mb_rank, *d_mb_pos;
  uint32_t *d_rank_mb_off, *d_rank_mbs, *d_rank_cnt, *d_tile_first_sample, *d_scalars;
  uint64_t *d_sample_cost, *d_mb_cost, *d_sample_row_off, *d_mb_row_off, *d_plan_len;
  uint64_t* d_row_src = nullptr;          // row words of the assembly (plans of written samples only)
  // Host-tier pages of the plan's own samples as copy-engine work: one entry per run of pages that follow one another
  // in a span's image and in the host slab, grouped by microbatch (entries of microbatch j: [mb_copy_off[j],
  // mb_copy_off[j+1])).  Made with the plan where the pool sends its host tier through the copy engine and no sample
  // of the plan is imported; a plan dies with the first free of one of its samples, so the pages cannot change.
  struct HostCopy {
    uint64_t row0;     // plan-global row of the span's first row
    uint64_t img_off;  // byte offset of the run in the span's image
    const void* src;   // host address of the run
    uint64_t len;
  };
  std::vector<HostCopy> host_copies;
  std::vector<uint32_t> mb_copy_off;
  bool host_copies_valid = false;
};

namespace ft {
inline PlanView make_plan_view(const ft_plan* pl) {
  PlanView pv;
  pv.n = pl->n; pv.n_mb = pl->n_mb; pv.n_ranks = pl->cfg.n_ranks_N;
  pv.mb_samples = pl->d_mb_samples; pv.plan_sample_mb = pl->d_plan_sample_mb;
  pv.sample_row_off = pl->d_sample_row_off; pv.mb_sample_off = pl->d_mb_sample_off;
  pv.mb_row_off = pl->d_mb_row_off; pv.tile_first_sample = pl->d_tile_first_sample;
  pv.row_src = pl->d_row_src;
  return pv;
}
// A plan dies with any of its samples (freed, or never completed under ALLOW_UNWRITTEN): FT_OK while every sample
// of the plan is READY in the generation the plan was made for, else FT_ERR_NOT_READY.
inline int32_t plan_alive(const ft_pool* p, const ft_plan* pl);
int32_t cuda_fail(cudaError_t e, const char* what);
// pools that exist (a plan may outlive its pool: plan_destroy must not touch a dead pool's block cache)
void pool_registry_add(ft_pool* p);
void pool_registry_remove(ft_pool* p);
bool pool_registry_has(ft_pool* p);
#define FT_CUDA(call)                                          \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    if (e__ != cudaSuccess) return ft::cuda_fail(e__, #call);  \
  } while (0)
}  // namespace ft

// ---- the pool's host object ----------------------------------------------------------------
enum { FT_SLOT_FREE = 0, FT_SLOT_REGISTERED = 1, FT_SLOT_READY = 2 };

struct ft_slot_mirror {
  uint8_t state = FT_SLOT_FREE;
  bool remote = false;  // imported from a peer: pages and text pages are not ours to recycle
  uint32_t seq_len = 0, n_spans = 0, spans_written = 0, n_text_pages = 0;
  uint64_t generation = 0;
  uint64_t named = 0;   // call_seq of the call that last listed this slot (duplicate detection inside one call)
};
struct ft_span_mirror {
  uint32_t pos = 0, tokens = 0, npages = 0;
  uint32_t grid[3] = {0, 0, 0};  // token grid (T, H, W) as last set; all zero = none
  bool written = false;
  uint64_t named = 0;   // call_seq of the write call that last named this span
  // the host's copy of the page list of an own written span: a chain through ft_pool::h_page_next (no allocation per write)
  uint32_t first_page = 0xFFFFFFFFu, owned_pages = 0;
};

// Per-call context: the descriptors of one ABI call travel host -> device through one of a small ring of these.
// `h` is pinned staging the call fills on the host; `d` is device scratch that receives the upload and the call's scan
// outputs; `counters` are two claim counters in the pool's metadata block (main and side stream of the call).  Two
// events guard reuse: the host waits for `ev_up` before it rewrites `h`; the metadata stream waits for `ev_done`
// (recorded behind the last kernel of the call that reads `d` or the counters) before it rewrites `d`.
struct ft_call_ctx {
  void* h = nullptr;   size_t hcap = 0;   void* hd = nullptr;  // `h` as the device sees it (mapped pinned memory)
  void* d = nullptr;   size_t dcap = 0;
  cudaEvent_t ev_up = nullptr, ev_done = nullptr;
  bool busy_up = false, busy_done = false;
  ft::ClaimCounter* counters = nullptr;  // [2], device
};
constexpr int kCallCtx = 16;

struct ft_pool {
  ft_pool_config cfg;
  ft::PoolView view;
  int device = 0;
  std::vector<ft_slot_mirror> slots;
  std::vector<ft_span_mirror> spans;  // [max_samples * spans_per_sample]
  uint64_t free_pages = 0, free_text_pages = 0, free_blocks = 0;
  uint64_t call_seq = 0, free_epoch = 0, live_samples = 0, live_spans = 0;
  uint64_t bytes_written = 0, bytes_gathered = 0, gpu_launches = 0;
  // allocations
  void* d_meta = nullptr;      // page tables, rings, tables, list blocks, status
  void* d_text = nullptr;      // text page frames
  void* hbm_base = nullptr;    bool own_hbm = false;
  void* host_base = nullptr;   bool own_host = false;  // host pointer
  void* host_dev = nullptr;                            // the same memory as the device sees it
  // per-call descriptors and scan outputs (see ft_call_ctx): one ring per side (0 = register, write, import, free,
  // span grids; 1 = plan, export, assemblies), so that a context of a long-running assembly is never the one a producer
  // call has to wait for
  ft_call_ctx ctx[2][kCallCtx];
  int ctx_next[2] = {0, 0};
  // The metadata stream.  Every kernel that only touches the pool's tables, rings and page lists (registration scan,
  // page allocation, the packing plan, free, import/export lists, span grids) runs here, in call order; the kernels
  // that move data (token ids, scatter, gather) run on the caller's stream behind an event of this one.  The
  // metadata of producer call i+1 is thus worked out while the scatter of call i streams, and the plan is made
  // while the last scatters run.
  cudaStream_t meta = nullptr;
  cudaEvent_t ev_meta = nullptr;      // re-recorded on `meta` whenever a caller's stream has to wait for it
  cudaEvent_t ev_in = nullptr;        // re-recorded on a caller's stream when `meta` has to wait for that stream
  cudaEvent_t ev_ids = nullptr;       // behind the latest copy of token ids into text pages (a caller's stream)
  bool have_ids_ev = false;
  cudaEvent_t ev_noalloc = nullptr;   // behind the last reader of the fixed no-allocation scratch
  bool have_noalloc_ev = false;
  uint64_t meta_seq = 0;              // metadata batches enqueued so far
  uint64_t ev_meta_seq = ~0ull;       // the batch count `ev_meta` was last recorded behind
  uint64_t status_base = 0;           // call_seq at the last pool_status read
  std::vector<uint8_t> noalloc_blob;  // host staging of pool_write_embeddings_noalloc, made at pool_create
  // Device blocks of destroyed plans, kept for the next plan: each with an event behind the last kernel that read it.
  // (A stream-ordered allocation would do, but a block freed on the stream of the last assembly and asked for again
  // on the metadata stream is not reusable across streams at once, and every other plan paid a fresh allocation.)
  struct plan_block { void* d; size_t cap; cudaEvent_t ev; };
  std::vector<plan_block> plan_cache;
  void* plan_pinned = nullptr;        // pinned landing zone of the plan's summary read-back (mapped: a kernel stores into it)
  void* plan_pinned_dev = nullptr;
  size_t plan_pinned_cap = 0;
  std::vector<uint32_t> bind_hbm, bind_host;           // vpn -> frame of this process's binding (exported to peers)
  // The host's copy of the FIFO page ring: pops and pushes are deterministic (calls in order, spans in argument order,
  // pages by ordinal), so the host can follow them and knows every span's pages without asking the device.  It serves
  // the copy-engine path of the host tier; the device's ring stays the one the kernels read.
  std::vector<uint32_t> h_ring;
  uint64_t h_ring_head = 0, h_ring_count = 0;
  std::vector<uint32_t> h_page_next;  // [pages] the page that follows in the same span's list
  int host_dma = 0;             // 1: host-tier pages of bf16 writes and of assemblies go through the copy engines
  void* d_text_base() const { return d_text; }
  std::vector<void*> peer_allocs;                      // imported peers' page-table arrays
  std::vector<uint8_t> peer_imported;                  // [world_size]
  bool peer_host_frames = false;                       // some imported peer binds host-tier pages
  bool peer_remote_frames = false;                     // some imported peer's HBM frames live on another GPU
  std::vector<std::array<uint64_t, 3>> peer_bases;     // [world_size] slab addresses (HBM, host, text) as seen here
  // host-tier traffic runs beside the HBM kernels on a side stream: one per side (0 producer, 1 consumer), so that
  // host-tier writes and host-tier reads of concurrent calls can use both directions of the link at once
  // (index 2: the consumer side's stream for frames in another GPU's HBM, read over NVLink)
  cudaStream_t side_stream[3] = {nullptr, nullptr, nullptr};
  cudaEvent_t fork_ev[3] = {nullptr, nullptr, nullptr}, join_ev[3] = {nullptr, nullptr, nullptr};
  // cross-stream ordering when the producer side and the consumer side are driven from different streams
  cudaEvent_t ev_producer = nullptr, ev_consumer = nullptr;  // end of the latest producer-side / consumer-side call
  bool have_producer_ev = false, have_consumer_ev = false;
  // samples in the order in which they became READY (slot, generation), for pool_take_ready
  std::deque<std::pair<uint32_t, uint64_t>> ready_fifo;
  int sm_count = 148;
  int occ_scatter[3][2] = {};   // resident CTAs/SM of k_scatter<tier mode, f32>, from the occupancy API
  int occ_gather[3][2] = {};    // resident CTAs/SM of k_gather<tier mode, U = 4 | 8>
  int host_ctas = 6;            // grid of the host-tier bulk-copy kernels: few SMs, so that long-latency host-link
                                // accesses do not clog the memory pipelines of the SMs that stream HBM; 6 rather
                                // than 8 because a write and a read kernel running together (two streams) share
                                // the link better with fewer requests in flight
  int scatter_smem_carveout = 5;  // percent of an SM's L1/shared storage the scatter kernel asks for as shared memory
  int gather_smem_carveout = 0;   // the same for the gather kernel (0 = the driver's choice)
  int remote_ctas = 16;         // grid of the bulk-copy gather from another GPU's HBM (about 128 KiB in flight per CTA;
                                // 770 GB/s x a few microseconds of NVLink latency wants 1.5 MB and more in flight)
  int peers_remote = 0;         // 1: flag every imported peer's HBM frames as remote, whatever device they are on
  int host_store_ctas = 8;      // grid of the vector-store scatter into host frames (fp32 sources, host-only pools)
  int chunk_shift = 0;          // log2 of k_scatter's work unit in bytes of a span's image (14..21); 0 = chosen per call
  int scatter_group = 0;        // chunks per round-robin group of k_scatter; 0 = the measured default
  int scatter_ctas_per_sm = 0;  // resident CTAs per SM of the device-tier scatter kernel; 0 = the measured default
  bool grad_attr_set = false;   // k_embed_grad_hot's shared-memory opt-in done
  int grad_hot_threshold = 0;   // rows from which an id takes k_embed_grad_hot; 0 = rows / (8 x grid), at least 64
  int grad_ctas_per_sm = 6;     // CTAs per SM of k_embed_grad (each owns the table rows v with v % grid == its index)
  int gather_unroll = 0;        // 16-byte vectors per lane in flight in k_gather (4 or 8); 0 = chosen per launch
  int dev_ctas_per_sm = 0;      // resident CTAs per SM of the device-tier gather kernel; 0 = chosen per launch
  // optional kernel timing (pool_profile_*)
  bool profiling = false;
  struct prof_rec { int kind; cudaEvent_t e0, e1; };
  std::vector<prof_rec> prof;
};

namespace ft {
// per-device set-up of each translation unit's kernels (shared-memory opt-ins, occupancy), run by pool_create
// with the pool's device current
int32_t gather_device_setup(ft_pool* p);
// shared-memory carve-out preference (percent) of the copy kernels of each translation unit
int32_t gather_set_carveout(int pct);
// n 32-bit words device <-> mapped host memory by a small kernel on `st` (not by a copy engine: see ctx_upload)
int32_t copy_words(void* dst, const void* src, size_t n_words, cudaStream_t st);
bool host_tier_by_copy_engine(const ft_pool* p);
// fills the plan's row words (metadata stream, behind the latest copy of token ids)
int32_t plan_rows_launch(ft_pool* p, ft_plan* pl);
int32_t scatter_set_carveout(int pct);
int32_t plan_device_setup(ft_pool* p);
// (d_list: device array of the list layout's entries, or nullptr for the range [mb_begin, mb_end))
int32_t gather_launch(ft_pool* p, const ft_plan* pl, uint32_t mb_begin, uint32_t mb_end, const void* embed_table,
                      uint32_t vocab, void* out_embeds, int32_t* out_cu, int32_t* out_pos, uint32_t pad_L, cudaStream_t st,
                      const void* d_list, uint32_t n_list, uint64_t list_tiles, uint64_t list_rows, ClaimCounter* counter,
                      const uint32_t* h_mb_list = nullptr);
__global__ void k_page_table_init(uint64_t* pte, const uint32_t* bind, uint64_t n, uint64_t base, uint64_t frame_bytes,
                                  uint64_t flags);
// uploads `bytes` from `src` (pageable) to the front of the pool's device scratch, asynchronously,
// through the staging ring; afterwards at least `total_bytes` of scratch exist.  Returns the device pointer.
// timing brackets around one kernel launch on `st` (no-ops unless profiling is on)
inline void prof_begin(ft_pool* p, int kind, cudaStream_t st) {
  if (!p->profiling) return;
  ft_pool::prof_rec r{kind, nullptr, nullptr};
  cudaEventCreate(&r.e0); cudaEventCreate(&r.e1);
  cudaEventRecord(r.e0, st);
  p->prof.push_back(r);
}
inline void prof_end(ft_pool* p, cudaStream_t st) {
  if (!p->profiling) return;
  cudaEventRecord(p->prof.back().e1, st);
}
size_t align_up_sz(size_t x, size_t a);
// Threads of a one-block scan kernel over n items: no more warps than there are items, so that the block fits on an
// SM beside the resident CTAs of a copy kernel (the metadata of one call is worked out while another call streams).
inline unsigned scan_threads(uint64_t n) { return (unsigned)(n >= 1024 ? 1024 : (n < 32 ? 32 : (n + 31) / 32 * 32)); }
// Takes the next call context: afterwards `h` holds at least `blob_bytes` of pinned staging the caller may fill, `d`
// at least `total_bytes` of device scratch no earlier kernel still reads (the metadata stream has been told to wait
// for the previous user; with on_meta = false it is `first_user` that waits, for a call that uploads nothing and
// only needs the context's counters on that stream).
// (side: 0 = producer-side calls, 1 = consumer-side calls)
int32_t ctx_acquire(ft_pool* p, int side, size_t blob_bytes, size_t total_bytes, ft_call_ctx** out, bool on_meta = true,
                    cudaStream_t first_user = nullptr);
// h[0, bytes) -> d[0, bytes) on the metadata stream
int32_t ctx_upload(ft_pool* p, ft_call_ctx* c, size_t bytes);
// `last` is the stream of the call's last kernel that reads the context
int32_t ctx_release(ft_pool* p, ft_call_ctx* c, cudaStream_t last);
// sequence number for asynchronous error keys of the current call
inline uint64_t status_seq(const ft_pool* p) { return (p->call_seq - p->status_base) & kStatusSeqMask; }
// `st` waits for everything enqueued on the metadata stream so far.  One event serves every stream that asks while no
// new metadata work is enqueued; once it has completed nobody needs to wait at all.  (No decision rests on the identity
// of a stream handle: a destroyed stream's handle may come back for a new stream.)
inline int32_t meta_to(ft_pool* p, cudaStream_t st) {
  if (p->ev_meta_seq != p->meta_seq) {
    FT_CUDA(cudaEventRecord(p->ev_meta, p->meta));
    p->ev_meta_seq = p->meta_seq;
  } else {
    const cudaError_t q = cudaEventQuery(p->ev_meta);
    if (q == cudaSuccess) return FT_OK;
    if (q != cudaErrorNotReady) return cuda_fail(q, "cudaEventQuery(ev_meta)");
  }
  FT_CUDA(cudaStreamWaitEvent(st, p->ev_meta, 0));
  return FT_OK;
}
// the metadata stream waits for everything enqueued on `st` so far
inline int32_t meta_after(ft_pool* p, cudaStream_t st) {
  FT_CUDA(cudaEventRecord(p->ev_in, st));
  FT_CUDA(cudaStreamWaitEvent(p->meta, p->ev_in, 0));
  return FT_OK;
}

// appends a sample that just became READY; entries of samples freed since are dropped whenever the queue has grown
// past four entries per slot, so a caller that never takes from it cannot make it grow without bound
inline void ready_push(ft_pool* p, uint32_t slot) {
  if (p->ready_fifo.size() > 4 * p->slots.size() + 64) {
    std::deque<std::pair<uint32_t, uint64_t>> live;
    for (const auto& e : p->ready_fifo)
      if (p->slots[e.first].state == FT_SLOT_READY && p->slots[e.first].generation == e.second) live.push_back(e);
    p->ready_fifo.swap(live);
  }
  p->ready_fifo.emplace_back(slot, p->slots[slot].generation);
}

// Cross-stream ordering.  Data kernels run on the callers' streams (a producer side and a consumer side, possibly two
// streams), metadata kernels on the pool's metadata stream:
//  * a consumer-side data kernel waits for the producer-side data kernels issued before it
//    and for the metadata enqueued so far;
//  * a metadata kernel that changes what data kernels already in flight may read (free, span grids) waits for the
//    latest producer-side and consumer-side data kernels;
//  * metadata kernels among themselves are ordered by the metadata stream.
inline int32_t begin_consumer(ft_pool* p, cudaStream_t st) {
  // (a wait for an event of the same stream costs nothing on the device; a completed event needs no wait)
  if (p->have_producer_ev && cudaEventQuery(p->ev_producer) != cudaSuccess) {
    cudaGetLastError();
    FT_CUDA(cudaStreamWaitEvent(st, p->ev_producer, 0));
  }
  return meta_to(p, st);
}
inline int32_t end_consumer(ft_pool* p, cudaStream_t st) {
  FT_CUDA(cudaEventRecord(p->ev_consumer, st));
  p->have_consumer_ev = true;
  return FT_OK;
}
// before metadata kernels that retire or change state data kernels in flight may still read
inline int32_t meta_after_data(ft_pool* p) {
  if (p->have_consumer_ev) FT_CUDA(cudaStreamWaitEvent(p->meta, p->ev_consumer, 0));
  if (p->have_producer_ev) FT_CUDA(cudaStreamWaitEvent(p->meta, p->ev_producer, 0));
  return FT_OK;
}
inline int32_t end_producer(ft_pool* p, cudaStream_t st) {
  FT_CUDA(cudaEventRecord(p->ev_producer, st));
  p->have_producer_ev = true;
  return FT_OK;
}
// The host-tier runs of an own span, from the host's copy of its page list: maximal sequences of pages that follow one
// another in the span's image and in the host slab.  fn(byte offset in the image, first frame, bytes).
template <class F>
inline void for_each_host_run(const ft_pool* p, const ft_span_mirror& m, uint64_t image_bytes, F&& fn) {
  const uint64_t PS = p->cfg.page_bytes, hbm = p->cfg.hbm_pages;
  uint32_t g = m.first_page;
  for (uint32_t k = 0; k < m.owned_pages;) {
    if (g < hbm) { g = p->h_page_next[g]; ++k; continue; }
    const uint64_t frame = p->bind_host[g - hbm];
    uint32_t k1 = k + 1, g1 = p->h_page_next[g];
    while (k1 < m.owned_pages && g1 >= hbm && p->bind_host[g1 - hbm] == frame + (k1 - k)) { g1 = p->h_page_next[g1]; ++k1; }
    const uint64_t off = (uint64_t)k * PS;
    fn(off, frame, (image_bytes < (uint64_t)k1 * PS ? image_bytes : (uint64_t)k1 * PS) - off);
    k = k1; g = g1;
  }
}
inline int32_t plan_alive(const ft_pool* p, const ft_plan* pl) {
  if (pl->free_epoch != p->free_epoch || (pl->cfg.flags & FT_PLAN_ALLOW_UNWRITTEN)) {
    for (uint32_t t = 0; t < pl->n; ++t) {
      const ft_slot_mirror& s = p->slots[pl->slots[t]];
      if (s.state != FT_SLOT_READY || s.generation != pl->slot_generation[t]) return FT_ERR_NOT_READY;
    }
  }
  return FT_OK;
}
}  // namespace ft
