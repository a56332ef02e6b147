/*
 * flowpool.h -- C ABI of the unified-memory-pool hot path on one B200 (sm_100a).
 *
 * The pool is the coordination layer between encoder producers and the LLM
 * backbone (paper Sec. 3.1-3.2): producers scatter embeddings into fixed-size
 * pages addressed by 64-bit global virtual addresses (GVAs); a page table maps
 * GVA -> physical frame in HBM or in pinned host DRAM; the dynamic packing
 * scheduler (Sec. 3.4, Algorithm 1, Eq. 3) forms balanced microbatches; the
 * consumer translates GVAs and assembles each packed microbatch.
 *
 * Conventions
 *  - Every call returns an int32 status: FT_OK or a negative FT_ERR_* code.
 *    Nothing throws, aborts or traps.
 *  - "host" / "device" in a parameter comment says where the pointer lives.
 *    Host arrays are read before the call returns.  `stream` is a cudaStream_t
 *    passed as void* (NULL = the legacy default stream).  Kernels that read or
 *    write the caller's data (token ids, embedding sources, the table, outputs)
 *    run on that stream, in stream order.  Kernels that only touch the pool's
 *    own tables, rings and page lists (registration scan, page allocation, the
 *    packing plan, free, import/export lists, span grids) run on a metadata
 *    stream the pool owns, in call order; the library links the two with
 *    events, so that every call still sees the effects of every earlier call
 *    of the pool, and whatever the caller enqueues on `stream` after a call
 *    comes after that call.  The gain: the page allocation of producer call
 *    i+1 is worked out while the copy of call i is streaming (Sec. 3.1: a
 *    producer goes on with its next batch at once).
 *  - Two streams per pool are supported: a producer side (register, write, import, free) and a consumer side
 *    (plan, export, gather) may be issued, from one host thread, on two different streams so that the encoder's
 *    scatter of the next batch overlaps the backbone's assembly of the current one (the decoupled
 *    producer-consumer flow of Sec. 3.1).  The library orders the sides itself: a consumer-side copy waits for
 *    the producer-side copies issued before it, and pool_free waits for the copies of both sides issued before it;
 *    the sides use separate call contexts and separate side streams for host-tier traffic.
 *  - A call may block the host briefly when the caller runs more than 8 calls of one side ahead of the device
 *    (the per-call descriptor staging is a ring of 16 pinned buffers per side).
 *  - One caller thread per pool.  The caller owns every buffer it passes in
 *    (backing memory, sources, table, outputs); the library owns its metadata
 *    and anything it allocated itself.
 *  - Errors the host can know (argument, state, capacity) are returned at once
 *    and the failed call has no effect (all-or-nothing; checks run in argument
 *    order, first failure wins).  Errors only the device can see go to an
 *    asynchronous status word read by pool_status(); the offending item is
 *    skipped.
 *  - The library needs a CUDA device; there is no CPU fallback.
 */
#ifndef FLOWPOOL_H_
#define FLOWPOOL_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  FT_OK = 0,
  FT_ERR_INVALID_ARG = -1,
  FT_ERR_POOL_EXHAUSTED = -2,
  FT_ERR_UNKNOWN_SAMPLE = -3,
  FT_ERR_ALREADY_WRITTEN = -4,
  FT_ERR_NOT_READY = -5,
  FT_ERR_TOO_LONG = -6,
  FT_ERR_BAD_GVA = -7,
  FT_ERR_PLACEHOLDER_MISMATCH = -8,
  FT_ERR_BAD_TOKEN_ID = -9,
  FT_ERR_SLOT_IN_USE = -10,
  FT_ERR_CAPACITY = -11,
  FT_ERR_CUDA = -12,
  FT_ERR_TIMEOUT = -13
};

enum { FT_RING_SORTED = 0, FT_RING_SHUFFLED = 1 }; /* initial free-ring order */
enum { FT_BIND_IDENTITY = 0, FT_BIND_PERMUTED = 1 }; /* virtual page -> frame */
enum { FT_BF16 = 0, FT_F32 = 1 };                    /* producer source dtype */
/* plan flags.  ALLOW_UNWRITTEN plans metadata only.  The others select variants at points where the paper
 * is silent or could be read otherwise (defaults follow the text): SORT_DECREASING packs longest first (equal
 * lengths keep the caller's order) instead of in the caller's order; COST_SUMSQ uses sum(l^2) instead of lmax^2
 * as the quadratic term of Eq. 3; ZIGZAG_CARRY lets the zig-zag position and direction carry over from bucket to
 * bucket instead of restarting in each; AUTO_K takes the number of buckets from the data, min(K, max(1,
 * ceil(n_mb / 2N))): one bucket per full zig-zag round trip over the N ranks, K being the upper limit. */
enum { FT_PLAN_ALLOW_UNWRITTEN = 1, FT_PLAN_SORT_DECREASING = 2, FT_PLAN_COST_SUMSQ = 4, FT_PLAN_ZIGZAG_CARRY = 8,
       FT_PLAN_AUTO_K = 16 };

#define FT_TEXT_PAGE_BYTES 4096u /* token ids live in 4 KiB text pages (1024 ids) */

typedef struct ft_pool ft_pool;
typedef struct ft_plan ft_plan;

/*
 * Pool geometry (Sec. 3.2).  The GVA space has two disjoint regions, one per
 * tier; region t is [start_t, start_t + world_size*max_size) and process i
 * owns [start_t + i*max_size, start_t + (i+1)*max_size).  This process binds
 * hbm_pages (resp. host_pages) frames of page_bytes at the base of its
 * segment; page k has GVA start_t + rank*max_size + k*page_bytes.  Text pages
 * follow the embedding pages inside the HBM segment.
 */
typedef struct {
  uint64_t page_bytes;      /* power of two, 4 KiB .. 2 MiB */
  uint64_t hbm_pages;       /* frames bound in HBM */
  uint64_t host_pages;      /* frames bound in pinned, device-mapped host DRAM */
  uint64_t max_text_tokens; /* text-page budget, in token ids (rounded up to whole text pages) */
  uint64_t ring_seed;       /* seed of FT_RING_SHUFFLED */
  uint64_t bind_seed;       /* seed of FT_BIND_PERMUTED (HBM: seed, host: seed+1) */
  uint64_t gva_hbm_start;   /* 0 => 2^44 */
  uint64_t gva_host_start;  /* 0 => 2^45 */
  uint64_t max_size;        /* per-process segment size; 0 => 2^40 */
  uint32_t hidden;          /* H, a multiple of 8 (a bf16 row is a multiple of 16 bytes) */
  uint32_t max_samples;     /* number of sample slots */
  uint32_t max_spans_per_sample;
  uint32_t max_pages_per_span;
  uint32_t max_seq_len;     /* longest sequence a slot may hold */
  int32_t placeholder_id;   /* the image-placeholder token id */
  uint32_t ring_order;      /* FT_RING_* */
  uint32_t bind_order;      /* FT_BIND_* */
  uint32_t world_size;      /* 0 => 1; processes of the GVA space (peers' bindings arrive by pool_import_mapping) */
  uint32_t rank;
  uint64_t max_imported_pages; /* list-block budget for samples imported from peers (their pages are not local) */
} ft_pool_config;

/* Packing parameters (Sec. 3.4): budget L, integer cost A*sum(l) + B*lmax^2
 * (Eq. 3 times L^2 when A = L, B = 1), K cost buckets, N data-parallel ranks. */
typedef struct {
  uint64_t coef_A, coef_B;
  uint32_t budget_L, n_buckets_K, n_ranks_N, flags;
} ft_plan_config;

typedef struct {
  uint64_t pages_total, pages_free, hbm_pages, host_pages;
  uint64_t text_pages_total, text_pages_free;
  uint64_t live_samples, live_spans;
  uint64_t bytes_written, bytes_gathered; /* algorithmic bytes enqueued so far */
  uint64_t gpu_launches;                  /* kernels of this library launched so far */
} ft_pool_stats;

/*
 * pool_create -- pool initialisation and binding (Sec. 3.2: each process
 * reserves a GVA range in its segment, allocates physical memory and binds it;
 * every process holds the page table locally).
 *   cfg      host.  See ft_pool_config.
 *   hbm_base device, caller-owned, >= hbm_pages*page_bytes, 256-byte aligned;
 *            NULL => the library allocates (and frees at pool_destroy).
 *   host_base host, caller-owned PINNED memory mapped into the device address
 *            space (cudaHostAlloc/cudaHostRegister with the mapped flag),
 *            >= host_pages*page_bytes; NULL => the library allocates.
 *   out      host; receives the handle.
 * Errors: INVALID_ARG (page_bytes not a power of two in range, hidden % 8,
 * no pages, segment too small, overlapping regions, rank >= world_size),
 * CUDA (allocation or launch failure).  Synchronises the device once.
 */
int32_t pool_create(const ft_pool_config* cfg, void* hbm_base, void* host_base, ft_pool** out);

/*
 * pool_register_samples -- text tokens and pairing metadata enter the pool
 * (Sec. 3.1: text tokens are inserted directly into the same pool; lightweight
 * metadata tracks the cross-modal pairing).  Sample i occupies slot
 * sample_slot[i]; its input_ids hold, for span j, one run of placeholder_id of
 * span_tokens[.] ids starting at span_pos[.] (sequence coordinates, sorted,
 * non-overlapping; spans of all samples concatenated in order).
 *   sample_slot, seq_len, n_spans  host [n]
 *   span_pos, span_tokens          host [sum n_spans]
 *   input_ids                      DEVICE int32 [sum seq_len], concatenated
 * Slot life cycle: FREE -> REGISTERED -> (all spans written) READY -> FREE.
 * Errors, per sample in order: slot >= max_samples INVALID_ARG; slot not FREE
 * or repeated SLOT_IN_USE; seq_len 0 INVALID_ARG; seq_len > max_seq_len or
 * n_spans > max_spans_per_sample CAPACITY; per span: 0 tokens, run past the
 * sequence, unsorted/overlapping runs INVALID_ARG, pages > max_pages_per_span
 * CAPACITY; then text pages exhausted CAPACITY.  Asynchronous: a run position
 * that is not placeholder_id or a stray placeholder -> PLACEHOLDER_MISMATCH
 * (detail = slot; the sample stays registered).
 */
int32_t pool_register_samples(ft_pool* pool, uint32_t n, const uint32_t* sample_slot,
                              const uint32_t* seq_len, const uint32_t* n_spans,
                              const uint32_t* span_pos, const uint32_t* span_tokens,
                              const int32_t* input_ids, void* stream);

/*
 * pool_write_embeddings -- the producer scatter (Sec. 3.1-3.2: encoders place
 * embeddings into their own segment and proceed at once).  Span q takes the
 * next ceil(n_tokens*2H/page_bytes) pages from the free ring, spans in
 * argument order; its bf16 row-major [n_tokens, H] image is laid into those
 * pages in order (rows may straddle pages; the last page's tail is untouched).
 *   sample_slot, span_idx, n_tokens  host [n_spans]
 *   src        host array [n_spans] of DEVICE pointers, each [n_tokens, H]
 *              contiguous, 16-byte aligned, FT_BF16 or FT_F32 elements
 *   src_dtype  FT_F32 fuses the fp32->bf16 cast: IEEE round-to-nearest-even
 *              on the bit pattern, denormals kept, every NaN -> sign | 0x7FC0.
 * Asynchronous: returns after enqueueing.  Errors, per span in order:
 * slot >= max_samples INVALID_ARG; slot FREE UNKNOWN_SAMPLE; span_idx out of
 * range, n_tokens != registered, src NULL or misaligned INVALID_ARG; span
 * written before or named twice ALREADY_WRITTEN; then sum of pages > free
 * pages POOL_EXHAUSTED.
 */
int32_t pool_write_embeddings(ft_pool* pool, uint32_t n_spans, const uint32_t* sample_slot,
                              const uint32_t* span_idx, const uint32_t* n_tokens,
                              const void* const* src, uint32_t src_dtype, void* stream);

/*
 * pool_write_embeddings_noalloc -- the same producer scatter for callers that must not allocate.
 * (The paper has no counterpart: this entry point exists for integration reasons only.)
 *
 * Who needs it: code that runs where a CUDA allocation is forbidden or would stall -- a producer thread
 * inside a region where the framework has frozen its allocator, a caller holding a memory budget it may
 * not exceed, a real-time loop that cannot afford the implicit device synchronisation of cudaMalloc/
 * cudaFree.  pool_write_embeddings may grow the pool's device scratch and its pinned staging buffers; this
 * variant never does.  It calls no cudaMalloc/cudaFree/cudaHostAlloc nor any other allocating routine:
 * the per-call descriptors and scan outputs (the only scratch memory the write path needs beyond its
 * inputs and the pool) live in one fixed array in the library's device image, FT_NOALLOC_SCRATCH_BYTES
 * long, which every GPU that loads the library holds until the process exits.
 *
 * Same arguments, result, status codes and check order as pool_write_embeddings, plus:
 *   - n_spans > FT_NOALLOC_MAX_SPANS -> FT_ERR_CAPACITY ("call too large for the fixed scratch"; split it);
 *   - the device current at the call must be the pool's device, else FT_ERR_INVALID_ARG.
 * The first call on each device looks up the array's device address once (cudaGetSymbolAddress); make
 * that first call before any stream capture begins.  All calls, from every pool on the device, share
 * the one array: it still holds the previous call's descriptors when the next call starts, and nothing in
 * it needs to start at zero except the two claim counters of the copy kernels in its last 32 bytes, which
 * the kernels themselves put back to zero when they finish.  A pool orders its own no-alloc writes (the
 * next one waits, on the GPU, for the copy of the one before); calls of DIFFERENT pools whose kernels may
 * overlap on the GPU race on the array -- give them one stream, or order them with events.
 * Host side: the descriptors are assembled in a buffer pool_create made for this purpose (the call needs
 * no more than a few hundred bytes of the caller's stack) and go up by cudaMemcpyAsync from that pageable
 * buffer, which returns only after the host data has been taken: the call blocks the host for that copy.
 */
#define FT_NOALLOC_MAX_SPANS 4096u
#define FT_NOALLOC_SCRATCH_BYTES (256u + 32u * (FT_NOALLOC_MAX_SPANS + 8u))
int32_t pool_write_embeddings_noalloc(ft_pool* pool, uint32_t n_spans, const uint32_t* sample_slot,
                                      const uint32_t* span_idx, const uint32_t* n_tokens,
                                      const void* const* src, uint32_t src_dtype, void* stream);

/*
 * pool_plan_microbatches -- the dynamic packing rule (Algorithm 1, Eq. 3), on
 * the device.  Samples are packed online in the order given, by best fit on
 * l(s) = seq_len (ties between equal residuals: the microbatch changed most
 * recently); each microbatch is scored A*sum(l) + B*lmax^2, bucketed by
 * equal-width quantisation of the observed cost range into K buckets, and
 * dealt zig-zag over N ranks per bucket (highest bucket first, cost
 * descending, ties by index).
 *   sample_slot host [n]; cfg host; out host, receives the plan handle.
 * Synchronises the stream once; the summary is valid on return.
 * cfg->flags may select the variants listed at FT_PLAN_*.
 * Errors: L, K or N zero INVALID_ARG; L >= 2^20 CAPACITY (the residual bitmap
 * covers budgets below 2^20); A*L + B*L^2 not representable in 64 bits
 * INVALID_ARG; per sample in order: slot out of range INVALID_ARG, FREE
 * UNKNOWN_SAMPLE, listed twice INVALID_ARG, not READY (without
 * FT_PLAN_ALLOW_UNWRITTEN) NOT_READY, seq_len > L TOO_LONG.
 * n = 0 gives an empty plan.
 */
int32_t pool_plan_microbatches(ft_pool* pool, const uint32_t* sample_slot, uint32_t n,
                               const ft_plan_config* cfg, ft_plan** out, void* stream);

/* Plan summary: number of microbatches, tokens over all of them, largest microbatch. */
int32_t plan_summary(const ft_plan* plan, uint32_t* n_mb, uint64_t* total_tokens,
                     uint32_t* max_mb_tokens);

/*
 * plan_arrays -- host copies of every plan array (any pointer may be NULL):
 * mb_sample_off[n_mb+1], mb_samples[n] (slots, microbatch-major, append
 * order), mb_tokens, mb_lmax, mb_residual, mb_cost (u64), mb_bucket,
 * mb_rank [n_mb], rank_mb_off[N+1], rank_mbs[n_mb] (dispatch order per rank),
 * sample_cost[n] (u64, Eq. 3 on a singleton), sample_mb[n].  Synchronises.
 */
int32_t plan_arrays(const ft_plan* plan, uint32_t* mb_sample_off, uint32_t* mb_samples,
                    uint32_t* mb_tokens, uint32_t* mb_lmax, uint32_t* mb_residual,
                    uint64_t* mb_cost, uint32_t* mb_bucket, uint32_t* mb_rank,
                    uint32_t* rank_mb_off, uint32_t* rank_mbs, uint64_t* sample_cost,
                    uint32_t* sample_mb);

/* Releases the plan.  Its device block is freed in stream order after the plan's latest work (no device-wide
 * synchronisation); the handle is invalid on return. */
int32_t plan_destroy(ft_plan* plan);

/*
 * pool_gather_packed -- the consumer (Sec. 3.1-3.2: the backbone consumes
 * microbatches by GVA; the GVA is resolved through the page table).  For
 * microbatches [mb_begin, mb_end) of the plan, concatenated: output row
 * cu_seqlens[q] + p of a microbatch is row (p - pos_start) of the span whose
 * placeholder run contains position p of its q-th sample, read through the
 * span's page list and the page table (HBM frame, or host frame read in place
 * over the mapped pointer); any other position is embed_table[input_ids[p]].
 *   embed_table       device bf16 [vocab, H]
 *   out_embeds        device bf16 [sum of tokens of the range, H], 16-byte aligned
 *   out_cu_seqlens    device int32, per microbatch (n_j + 1) entries starting at 0
 *   out_position_ids  device int32 [sum of tokens]: p, restarting per sample
 * Padding rows are not materialised.  Asynchronous.  Errors: bad range
 * INVALID_ARG; a sample of the plan freed or not READY NOT_READY; NULL buffer
 * INVALID_ARG; hidden > 18432 CAPACITY (a row may touch at most 10 pages).
 * Asynchronous: id outside [0, vocab) BAD_TOKEN_ID, page GVA that does not
 * translate BAD_GVA (detail = row index in the range; row skipped).  Whether a
 * position is a vision row is decided by the sample's span table, not by its id.
 */
int32_t pool_gather_packed(ft_pool* pool, const ft_plan* plan, uint32_t mb_begin, uint32_t mb_end,
                           const void* embed_table, uint32_t vocab, void* out_embeds,
                           int32_t* out_cu_seqlens, int32_t* out_position_ids, void* stream);

/*
 * pool_gather_list -- pool_gather_packed for a list of microbatches instead of a range (Algorithm 1 deals
 * microbatches to ranks, lines 15-27: a rank's share, `rank_mbs` of plan_arrays, is not contiguous).  Outputs are
 * the concatenation, in list order, of what pool_gather_packed writes for each [j, j+1): rows, n_j + 1
 * cu_seqlens entries per listed microbatch, position ids.  One launch per tier for the whole list.
 *   mb_list host [n_list]; an index may repeat.
 * Errors: index >= n_mb INVALID_ARG; otherwise as pool_gather_packed (asynchronous errors: detail = row index in
 * this call's output).  Asynchronous.
 */
int32_t pool_gather_list(ft_pool* pool, const ft_plan* plan, const uint32_t* mb_list, uint32_t n_list,
                         const void* embed_table, uint32_t vocab, void* out_embeds, int32_t* out_cu_seqlens,
                         int32_t* out_position_ids, void* stream);

/*
 * pool_free -- release samples: their pages go back to the free-ring tail
 * (samples in argument order, spans by index, pages by ordinal), their text
 * pages and slots are recycled.  Plans holding a freed sample become invalid.
 * The paper does not discuss recycling; the FIFO ring is this library's fixed rule.
 *   sample_slot host [n].  Errors: slot out of range INVALID_ARG; FREE or
 * listed twice UNKNOWN_SAMPLE.  Asynchronous.
 */
int32_t pool_free(ft_pool* pool, const uint32_t* sample_slot, uint32_t n, void* stream);

/*
 * FT_ERR_TIMEOUT is the one asynchronous error that is not about the caller's data.  The host-tier kernels move pages
 * with bulk-asynchronous copies and wait for each staged load on an mbarrier; that wait, the library's only device-side
 * spin, gives up after 2 s of wall clock (a host link that has stopped answering; ft_tuning.bulk_wait_limit_us).  The
 * CTA then issues no further copy, waits once more -- again at most that long -- for the loads it had already issued,
 * and returns; detail = CTA index (low 16 bits) | loads that had still not arrived when it returned (high 16 bits; 0
 * means that none can land later).  The bytes of that call are incomplete and the pool's state is no longer
 * trustworthy: after FT_ERR_TIMEOUT the only call a pool still supports is pool_destroy.  (Under the test hook
 * ft_tuning.bulk_timeout_test nothing was lost: the call's output is incomplete, the pool is intact.)
 */
/* First asynchronous error since the last call of pool_status (smallest call, then smallest code, then smallest
 * detail), then cleared.  Synchronises the device.  Calls are numbered from the last read, on 28 bits: read the
 * status at least once every 2^28 calls of the pool (a training run that checks it once per step never comes close). */
int32_t pool_status(ft_pool* pool, int32_t* first_device_error, uint64_t* detail);

int32_t pool_stats(ft_pool* pool, ft_pool_stats* out);

/*
 * Ready queue (Sec. 3.1: the scheduler forms microbatches once enough paired embeddings are in the pool).
 * Samples enter a FIFO in the order in which they became READY (last span written, text-only registration, import).  pool_ready_count reports the live entries and their tokens.  pool_take_ready pops up
 * to max_samples slots in that order, but only once at least min_tokens tokens are ready (the watermark):
 * otherwise NOT_READY and nothing is taken.  Entries of samples freed in the meantime are skipped.  Host only.
 */
int32_t pool_ready_count(ft_pool* pool, uint32_t* n_samples, uint64_t* n_tokens);
int32_t pool_take_ready(ft_pool* pool, uint64_t min_tokens, uint32_t max_samples, uint32_t* slots_out /* host */,
                        uint32_t* n_out, uint64_t* tokens_out);

/*
 * More than one process in the GVA space (Sec. 3.2: every process sends its memory mapping to all the others, which
 * enter it into their page tables; afterwards address translation is local).
 * Pools created with the same world_size, page_bytes, GVA starts and max_size and distinct ranks form one space.
 *
 * pool_backing        the addresses of this pool's slabs as THIS process sees them (device pointers; the host
 *                     slab as the device sees it).  A peer in another process needs its own view of them (an IPC
 *                     or fabric mapping); in one process, with peer access enabled, these are usable as they are.
 * pool_export_mapping this process's binding (geometry + vpn->frame of both tiers) into a host buffer.
 *                     buf = NULL queries the size.  CAPACITY if cap is too small.
 * pool_import_mapping installs a peer's binding: builds that process's page-table arrays from the blob and the
 *                     three base addresses at which this device reaches the peer's HBM slab, host slab and text
 *                     frames.  HBM frames of a slab that lives on another GPU are flagged remote (the transport is
 *                     chosen by where source and destination are, Sec. 3.2): assemblies read them with a separate,
 *                     small bulk-copy launch beside the one that streams local HBM.  INVALID_ARG: malformed blob, another GVA space, own rank, missing or misaligned
 *                     base; SLOT_IN_USE: that rank was imported before.  Init-time: allocates, synchronises.
 * pool_export_samples descriptors of READY samples (lengths, spans with their token grids, page GVAs, text-page GVAs) into a host buffer
 *                     -- the small metadata records a consumer needs; no embedding bytes.  Synchronises `stream`.
 *                     UNKNOWN_SAMPLE / NOT_READY / INVALID_ARG (repeated slot) per sample in order; buf = NULL
 *                     queries the size.
 * pool_import_samples registers the described samples in local FREE slots as READY, imported samples: their page
 *                     lists point into the peer's segment and are read in place by pool_gather_packed; they take
 *                     list blocks but no pages here, and pool_free returns nothing to the page rings for them.
 *                     The producer must keep the samples alive until the consumer has freed its imports.
 *                     INVALID_ARG: malformed blob or the source rank's mapping not imported; SLOT_IN_USE;
 *                     CAPACITY: a sample exceeds this pool's limits or the list blocks run out.  Asynchronous.
 */
int32_t pool_backing(ft_pool* pool, void** hbm_base, void** host_base_device, void** text_base);

/*
 * Peers in other processes of the same node.  pool_ipc_export fills shareable handles (CUDA IPC) of the HBM slab
 * and the text frames this pool allocated (INVALID_ARG for a caller-owned HBM slab: share that yourself);
 * pool_ipc_open, called in the consumer's process, maps them and returns the base addresses to hand to
 * pool_import_mapping; pool_ipc_close unmaps them (after the imported samples were freed).  The handle bytes travel
 * by any host channel, next to the mapping blob.  Host-tier pages of another process are reached through a
 * pointer the caller provides (shared host memory registered with the device); these calls do not cover them.
 */
#define FT_IPC_HANDLE_BYTES 64
typedef struct {
  uint8_t hbm[FT_IPC_HANDLE_BYTES], text[FT_IPC_HANDLE_BYTES];
  uint32_t has_hbm, has_text;
} ft_ipc_handles;
int32_t pool_ipc_export(ft_pool* pool, ft_ipc_handles* out);
int32_t pool_ipc_open(const ft_ipc_handles* in, void** hbm_base, void** text_base);
int32_t pool_ipc_close(void* hbm_base, void* text_base);
int32_t pool_export_mapping(ft_pool* pool, void* buf /* host */, uint64_t cap, uint64_t* bytes);
int32_t pool_import_mapping(ft_pool* pool, const void* buf /* host */, uint64_t bytes, void* peer_hbm_base,
                            void* peer_host_base, void* peer_text_base);
int32_t pool_export_samples(ft_pool* pool, const uint32_t* sample_slot, uint32_t n, void* buf /* host */, uint64_t cap,
                            uint64_t* bytes, void* stream);
int32_t pool_import_samples(ft_pool* pool, const uint32_t* local_slot, uint32_t n, const void* buf /* host */,
                            uint64_t bytes, void* stream);

/*
 * Backbone-side outputs next to assembly.  The paper stops where the backbone consumes a microbatch (Sec. 3.1);
 * no passage defines what follows, so the definitions are stated here.  They lean on three facts the paper does
 * fix: image and text subsequences are interleaved (Sec. 4.1), a microbatch holds at most L tokens (Sec. 3.4),
 * and the encoders are frozen, so the only gradient that flows back through the assembled input is the
 * embedding table's.
 *
 * pool_set_span_grids -- token grid (T, H, W) of named spans, T*H*W = the span's tokens, tokens in row-major
 * (t, h, w) order.  A span keeps its grid until its sample is freed; a span without one counts as text below; of
 * several items naming the same span the last one stays.
 *   slot, span_idx host [n]; grid_thw host [n][3].  All-or-nothing, first bad item in order: slot out of range
 *   INVALID_ARG, FREE slot UNKNOWN_SAMPLE, no such span INVALID_ARG, a zero extent or a product that is not the
 *   span's token count INVALID_ARG.  Asynchronous; ordered before later calls on any stream like a producer call.
 */
int32_t pool_set_span_grids(ft_pool* pool, uint32_t n, const uint32_t* slot, const uint32_t* span_idx,
                            const uint32_t* grid_thw, void* stream);

/*
 * pool_gather_padded -- pool_gather_packed in the padded layout: microbatch j of [mb_begin, mb_end) occupies rows
 * [(j - mb_begin) * L, (j - mb_begin + 1) * L) of every output, L the plan's budget; rows = (mb_end - mb_begin) * L.
 *   out_embeds   device bf16 [rows, H], 16-byte aligned: the packed rows of the microbatch, then zero rows
 *   out_cu       device int32, per microbatch n_j + 2 entries: 0, the sample ends, then L (the padding as one
 *                last sequence, of length 0 when the microbatch is full)
 *   out_pos3     device int32 [3, rows], component-major.  A counter st runs over each sample from 0: a text token
 *                (or a token of a span without a grid) gets (st, st, st) and st += 1; a span with grid (T, H, W)
 *                starting at counter st gives its token (t, h, w) the position (st + t, st + h, st + w), then
 *                st += max(T, H, W).  0 on padding rows.  Without any grid all three equal the packed position ids.
 *   out_ids      device int32 [rows]: the stored token id of the position (the placeholder id inside a span);
 *                pad_id on padding rows
 *   out_labels   device int32 [rows]: next-token target: the id at the next position of the same sample when
 *                that position is a text position, else -100; -100 on a sample's last position and on padding
 *   out_mask     device uint8 [rows]: 1 where the label is not -100
 * Errors as pool_gather_packed (detail = padded row index); more than 2^32 - 1 padded rows CAPACITY.  Asynchronous.
 */
int32_t pool_gather_padded(ft_pool* pool, const ft_plan* plan, uint32_t mb_begin, uint32_t mb_end,
                           const void* embed_table, uint32_t vocab, int32_t pad_id, void* out_embeds,
                           int32_t* out_cu, int32_t* out_pos3, int32_t* out_ids, int32_t* out_labels,
                           uint8_t* out_mask, void* stream);

/*
 * pool_embed_grad -- gradient of the embedding table through the assembled input.  grad_out holds one bf16 row
 * per output row of the range, in the packed layout (padded = 0) or the padded layout (padded != 0).  For the
 * rows in ascending order: a row at a text position with id v adds its values, widened exactly to fp32, to row v
 * of grad_table, one rounded fp32 addition per element; rows at span positions and padding rows add nothing.
 * The order of the additions is part of the definition (fp32 addition is not associative): results are
 * bit-reproducible and independent of the launch geometry.
 *   grad_out    device bf16 [rows, H], 16-byte aligned
 *   grad_table  device fp32 [vocab, H], 16-byte aligned, accumulated in place
 * Errors: as pool_gather_packed; asynchronous: id outside [0, vocab) BAD_TOKEN_ID (row skipped).  Allocates
 * stream-ordered scratch for the call (about 24 bytes per row plus 8 bytes per table row).  Ids that own many
 * rows are added by a separate kernel on the pool's second consumer-side stream; the call returns with `stream`
 * ordered after both.
 */
int32_t pool_embed_grad(ft_pool* pool, const ft_plan* plan, uint32_t mb_begin, uint32_t mb_end, uint32_t padded,
                        const void* grad_out, float* grad_table, uint32_t vocab, void* stream);

/*
 * Kernel timing for benchmarks.  While enabled, the library brackets each of its copy kernels with CUDA
 * events on the stream that kernel is launched on (the host-tier kernels run on the pool's side stream).
 * pool_profile_read synchronises the device, adds up the elapsed time and launch count per kernel class
 * since the last read, and clears them.  Classes: a single-tier pool's kernels count under its tier.
 */
enum { FT_K_GATHER_DEVICE = 0, FT_K_GATHER_HOST = 1, FT_K_SCATTER_DEVICE = 2, FT_K_SCATTER_HOST = 3, FT_K_EMBED_GRAD = 4,
       FT_K_GATHER_REMOTE = 5, FT_K_COUNT = 6 };
typedef struct {
  double ms;
  uint64_t launches;
} ft_kernel_time;
int32_t pool_profile_enable(ft_pool* pool, int32_t on);
int32_t pool_profile_read(ft_pool* pool, ft_kernel_time* out /* host [FT_K_COUNT] */);

/*
 * Launch geometry of the data kernels.  The paper has no counterpart: these are this library's knobs, all of them
 * in this one struct (nothing is read from the environment).  pool_get_tuning returns the values in force;
 * pool_set_tuning replaces them (0 in a field = that field's built-in default, the optimum measured on a B200);
 * out-of-range values INVALID_ARG and nothing changes.  Call it between other calls of the pool; it synchronises
 * the device.  None of the knobs changes any result (bulk_timeout_test, a test hook, excepted).
 *   dev_ctas_per_sm      resident CTAs per SM of the HBM-tier gather kernel (1..8).  Default 0 = chosen per launch
 *                        together with gather_unroll: 4 CTAs x 4 vectors for a range of one wave or rows under 4 KiB,
 *                        2 CTAs x 8 vectors for longer ranges
 *   scatter_ctas_per_sm  resident CTAs per SM of the HBM-tier scatter kernel (default 4; 1..8)
 *   scatter_group        chunks a scatter CTA claims at a time (default 1)
 *   chunk_shift          log2 of the scatter's work unit in bytes of a span's image (14..21).  Default 0 = chosen per
 *                        call: 16 KiB chunks while the call has at most 2^17 of them, else 32 KiB, else 64 KiB (small
 *                        chunks shorten the last wave of a launch; each chunk has a 24-byte record in the call's
 *                        scratch where pages are at least a chunk long)
 *   host_ctas            grid of the host-tier bulk-copy kernels (default 6): few SMs, so that long-latency host-link
 *                        accesses do not clog the memory pipelines of the SMs that stream HBM
 *   host_store_ctas      grid of the vector-store scatter into host frames (fp32 sources, host-only pools; default 8)
 *   gather_unroll        16-byte vectors per lane in flight in the gather kernel (4 or 8; default 0 = see above)
 *   grad_ctas_per_sm     CTAs per SM of the table-gradient kernel (default 6; 1..8)
 *   grad_hot_threshold   rows from which an id takes the frequent-id gradient kernel (default rows / (8 x grid), >= 64)
 *   remote_ctas          grid of the bulk-copy gather that reads frames in ANOTHER GPU's HBM (default 16): like the
 *                        host tier, peer frames are long-latency sources and get a small grid of their own, so that the
 *                        SMs that stream local HBM keep their memory pipelines; to be tuned where a second GPU exists
 *   scatter_smem_carveout  shared-memory share, in percent of an SM's unified L1/shared storage, that the scatter
 *                        kernel asks for although it uses next to none (default 5; 1..100; a function attribute, so
 *                        it holds for the device, not only for this pool).  An SM keeps one split while any CTA is
 *                        resident.  With the driver's own choice for this kernel the metadata kernels and the packing
 *                        kernel did not start beside it and ran when the copies had ended; with 3 to 9 percent they
 *                        run beside it and the copy streams as fast as before; from 10 percent on the copy loses a
 *                        sixth of its bandwidth (measured on a B200)
 *   gather_smem_carveout   the same preference for the gather kernel (default 0 = the driver's choice: this kernel
 *                        keeps 6 KiB of row descriptors per CTA in shared memory, and a preference below what four
 *                        CTAs need costs it occupancy and 6 percent of its bandwidth)
 *   peers_remote         1: pool_import_mapping flags every peer's HBM frames as remote even when they are on this
 *                        device (exercises the remote path on one GPU); 0: only frames of another device are remote
 *   host_copy_engine     who moves host-tier pages of bf16 writes and of assemblies.  0 (default): the bulk-copy
 *                        kernels.  1: the copy engines: one cudaMemcpyAsync per run of pages that are contiguous in a
 *                        span's image and in the host slab, issued from the host's own copy of the page lists (fp32
 *                        sources, imported samples and plans made under the other setting still take the kernels).
 *                        Measured on a B200 host: single 2 MiB pages move as fast either way (50 GB/s), runs of 8 MiB
 *                        and more reach the link's rate (54-55 GB/s against 46-51), which a pool with an identity
 *                        binding gets (config 2: 717 against 645 GB/s for the whole step).  The price: a copy
 *                        engine serves its queue in order, so these copies wait behind any bulk copy the application
 *                        has queued in the same direction, and the application's behind them; the kernels share
 *                        the link but no queue.  Hence off by default
 *   bulk_wait_limit_us   bound, in microseconds, of every wait of the bulk-copy kernels for a staged load (default
 *                        2 000 000; 100..10 000 000).  A load not seen within it is declared lost and the call
 *                        reports FT_ERR_TIMEOUT through the status word (see FT_ERR_TIMEOUT above)
 *   bulk_timeout_test    test hook for that path, 0 in use.  1: every staged load announces 16 bytes more to its
 *                        completion barrier than it requests, so that no load is ever SEEN complete although all of
 *                        them arrive: each bulk-copy CTA runs its first wait to the limit, gives up, waits once more
 *                        (bounded) for the loads it had issued, and returns; the call stores nothing from those
 *                        frames and reports FT_ERR_TIMEOUT.  Nothing faults and nothing spins beyond twice the
 *                        limit; accepted only with bulk_wait_limit_us set to at most 100 000.  This is the one knob
 *                        that changes results
 */
typedef struct {
  uint32_t dev_ctas_per_sm, scatter_ctas_per_sm, scatter_group, chunk_shift;
  uint32_t host_ctas, host_store_ctas, gather_unroll, grad_ctas_per_sm, grad_hot_threshold;
  uint32_t remote_ctas, peers_remote, scatter_smem_carveout, gather_smem_carveout;
  uint32_t bulk_wait_limit_us, bulk_timeout_test;
  uint32_t host_copy_engine;
} ft_tuning;
int32_t pool_get_tuning(ft_pool* pool, ft_tuning* out);
int32_t pool_set_tuning(ft_pool* pool, const ft_tuning* in);

/* Page GVAs of one span, by ordinal (for parity checks).  Synchronises. */
int32_t pool_debug_span_pages(ft_pool* pool, uint32_t slot, uint32_t span, uint64_t* gva_out,
                              uint32_t cap, uint32_t* n);

/* Free ring content, head first, as global page indices.  Synchronises. */
int32_t pool_debug_ring(ft_pool* pool, uint32_t* out, uint64_t cap, uint64_t* n);

/* Device-side GVA translation of a host array of GVAs (for parity checks):
 * kind 0 HBM / 1 host / 2 text, frame index within its tier, byte offset;
 * status[i] = FT_OK or FT_ERR_BAD_GVA.  Synchronises. */
int32_t pool_debug_translate(ft_pool* pool, const uint64_t* gva, uint32_t n, uint32_t* kind,
                             uint64_t* frame, uint64_t* offset, int32_t* status);

/* Tear down: frees everything the library allocated.  Synchronises. */
int32_t pool_destroy(ft_pool* pool);

/* Last CUDA error string seen by this library on the calling thread (thread-local storage: with one caller
 * thread per pool, that is the pool's own last error). */
const char* flowpool_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FLOWPOOL_H_ */
