// The consumer: GVA translation and packed-microbatch assembly (Sec. 3.1-3.2).
//
// k_gather: output rows are cut into units of up to 32 consecutive rows, claimed in order from a device counter.
// Each CTA has one resolver warp and eight streaming warps.  The resolver works one unit ahead: while the streaming
// warps copy unit t with 16-byte vectors, it claims unit t+1 and resolves its row sources, one lane per row (plan
// position -> slot -> token id from the text page; a placeholder position -> span -> page ordinal -> page GVA from
// the span's two-level list -> page-table entry), leaving the frame addresses in the other half of a double buffer
// in shared memory.  Rows that straddle pages carry one address per page touched.  With a two-tier pool the kernel
// is launched once per tier, so host-link reads never stall HBM reads.
//
// Row table.  A plan of written samples carries one 64-bit word per output row, made once when the plan is made
// (k_plan_rows): position in the sample plus the token id (text row) or the span (placeholder row).  With it the
// resolver's chain of dependent loads is claim -> row word -> table row (text) or -> page list -> page-table entry
// (vision) instead of eight to ten steps; it matters where a CTA resolves its first unit with nothing to overlap it
// (short ranges: one microbatch per call, the tiny configuration).  The table holds no address and no page: a row
// whose word says "unresolved" (0) takes the long way, so results and errors are the same with and without it.
#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <type_traits>
#include <vector>

#include "bulk_copy.cuh"
#include "flowpool_internal.cuh"

namespace ft {

constexpr int kTileRows = 32;
constexpr int kMaxSeg = 10;  // pages one row can touch: row_bytes <= 32 KiB over 4 KiB pages, plus a straddle
constexpr int kStreamWarps = 8;                          // warps that copy rows
constexpr int kGatherThreads = 32 * (kStreamWarps + 1);  // + the resolver warp

enum { kTierAll = 0, kTierDeviceOnly = 1, kTierHostOnly = 2 };

// row word: kind (2 bits: 0 unresolved, 1 text, 2 placeholder) | position in the sample (30 bits) | token id or span id
constexpr uint64_t kRowText = 1ull << 62, kRowVision = 2ull << 62;

struct RowDesc {
  uint64_t seg[kMaxSeg];  // page-table entries (frame address | flags) of the pages the row touches
  uint32_t off0;          // byte offset of the row inside its first page (0 for a text row)
  uint32_t shift;         // log2(page bytes); 31 for a text row (one segment)
  uint32_t nseg;          // 0 = nothing to copy
  uint32_t out_row;       // output row of this row (range, padded or list layout)
};

// One listed microbatch (list layout): its plan rows, where its tiles start in the claim order, where its output starts.
struct ListEntry {
  uint64_t row_lo, row_hi;  // plan-global rows
  uint64_t tile0;           // claim index of its first tile
  uint64_t out_row0;        // first output row
  uint32_t q_lo, q_hi;      // plan positions of its samples
  uint32_t cu0, pad;        // first cu_seqlens entry
};

struct GatherArgs {
  uint32_t q_lo, q_hi, mb_begin;  // plan positions and first microbatch of the range
  uint64_t row_lo, row_hi;        // plan-global output rows of the range
  const uint8_t* table;
  uint32_t vocab;
  uint8_t* out;
  int32_t* cu;
  int32_t* pos_ids;
  uint64_t call_seq;
  uint32_t write_index;  // this launch writes cu_seqlens / position ids
  uint32_t pad_L;        // 0: packed rows; else every microbatch starts at a multiple of pad_L rows (padded layout)
  uint32_t sub_shift;    // a claim covers 32 >> sub_shift rows (short ranges are cut finer, so that every SM has work)
  ClaimCounter* tile_counter;  // device, zero at rest
  const ListEntry* list;             // list layout: the microbatches to assemble, in output order (else nullptr)
  uint32_t n_list;
  uint64_t list_tiles;               // tiles over all entries
};

template <int MODE, int U, bool LIST>
__global__ void __launch_bounds__(kGatherThreads) k_gather(PoolView v, PlanView pl, GatherArgs a) {
  __shared__ RowDesc desc[2][kTileRows];
  __shared__ uint32_t valid[2];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint64_t tile_lo = a.row_lo / kTileRows, tile_hi = (a.row_hi + kTileRows - 1) / kTileRows;
  const uint32_t row_vecs = v.row_bytes >> 4;
  const uint32_t R = kTileRows >> a.sub_shift, sub_mask = (1u << a.sub_shift) - 1;
  const bool resolver = warp == kStreamWarps;

  // Resolver warp: claims the next unit (units are claimed in order, so the CTAs in flight always cover one compact
  // window of the output and uneven units balance themselves; a CTA's first unit is its block index, which saves one
  // round trip to the counter) and resolves its rows into desc[buf].
  const bool use_rows = pl.row_src != nullptr && a.pad_L == 0;
  bool first_claim = true;
  // cu_seqlens of a sample whose first row was resolved through the row table: written after the unit is published
  uint64_t pend_row = ~0ull, pend_cu0 = 0;
  uint32_t pend_q_lo = 0, pend_tile_q = 0;
  auto finish_index = [&]() {
    if (pend_row == ~0ull) return;
    uint32_t q = pend_tile_q;
    if (q < pend_q_lo) q = pend_q_lo;
    while (pend_row >= pl.sample_row_off[q + 1]) ++q;
    const uint32_t j = pl.plan_sample_mb[q];
    const uint64_t e = LIST ? pend_cu0 + (q - pend_q_lo) : (uint64_t)(q - a.q_lo) + (j - a.mb_begin);
    a.cu[e] = (int32_t)(pl.sample_row_off[q] - pl.mb_row_off[j]);
    if (q + 1 == pl.mb_sample_off[j + 1]) a.cu[e + 1] = (int32_t)(pl.sample_row_off[q + 1] - pl.mb_row_off[j]);
    pend_row = ~0ull;
  };
  auto resolve = [&](uint32_t buf) {
    unsigned long long c = 0;
    if (first_claim) {
      c = blockIdx.x;
      first_claim = false;
    } else {
      if (lane == 0) c = gridDim.x + atomicAdd(&a.tile_counter->claim, 1ull);
      c = __shfl_sync(0xFFFFFFFFu, c, 0);
    }
    const uint64_t ct = c >> a.sub_shift;  // claim index in whole 32-row tiles
    uint64_t tile = ~0ull;
    uint32_t entry = 0;
    if (LIST) {
      // list layout: the entry holding the claim (last entry whose first tile is <= ct), then its plan tile
      uint32_t lo = 0, hi = a.n_list;
      while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (a.list[mid].tile0 <= ct) lo = mid; else hi = mid;
      }
      entry = lo;
      if (ct < a.list_tiles) tile = a.list[lo].row_lo / kTileRows + (ct - a.list[lo].tile0);
    } else if (tile_lo + ct < tile_hi) {
      tile = tile_lo + ct;
    }
    if (tile == ~0ull) {  // past the end: this CTA is done claiming
      if (lane == 0) { valid[buf] = 0; claim_release(a.tile_counter); }
      return;
    }
    if (lane == 0) valid[buf] = 1;
    if (lane >= R) return;
    const uint64_t row = tile * kTileRows + (uint64_t)((uint32_t)c & sub_mask) * R + lane;
    RowDesc d;
    d.nseg = 0; d.off0 = 0; d.shift = 31; d.out_row = 0;
    // the rows this unit may touch: the call's range, or the listed microbatch it belongs to
    uint64_t row_lo = a.row_lo, row_hi = a.row_hi, out0 = 0, cu0 = 0;
    uint32_t q_lo = a.q_lo;
    if (LIST) {
      const ListEntry en = a.list[entry];
      row_lo = en.row_lo; row_hi = en.row_hi; out0 = en.out_row0; cu0 = en.cu0; q_lo = en.q_lo;
    }
    if (row >= row_lo && row < row_hi) {
      const uint64_t word = use_rows ? pl.row_src[row] : 0ull;
      uint32_t p, sid = 0;
      uint64_t out_row = out0 + (row - row_lo);
      int kind = (int)(word >> 62);  // 0: the long way
      int32_t id = -1;
      bool text_ok = true;
      if (kind) {
        p = (uint32_t)(word >> 32) & 0x3FFFFFFFu;
        if (kind == 1) id = (int32_t)(uint32_t)word; else sid = (uint32_t)word;
        if (a.write_index) {
          a.pos_ids[out_row] = (int32_t)p;
          if (p == 0) { pend_row = row; pend_cu0 = cu0; pend_q_lo = q_lo; pend_tile_q = pl.tile_first_sample[tile]; }
        }
      } else {
        // plan position of the sample holding this row: the tile's first sample, then a short walk
        uint32_t q = pl.tile_first_sample[tile];
        if (q < q_lo) q = q_lo;
        while (row >= pl.sample_row_off[q + 1]) ++q;
        p = (uint32_t)(row - pl.sample_row_off[q]);
        const uint32_t slot = pl.mb_samples[q];
        if (!LIST && a.pad_L) {  // padded layout: microbatch j of the range starts at row (j - mb_begin) * L
          const uint32_t j = pl.plan_sample_mb[q];
          out_row += (uint64_t)(j - a.mb_begin) * a.pad_L - (pl.mb_row_off[j] - a.row_lo);
        }
        if (a.write_index) {
          a.pos_ids[out_row] = (int32_t)p;
          if (p == 0) {  // cu_seqlens: every sample writes its start; the last of a microbatch also the end
            const uint32_t j = pl.plan_sample_mb[q];
            const uint64_t e = LIST ? cu0 + (q - q_lo) : (uint64_t)(q - a.q_lo) + (j - a.mb_begin);
            a.cu[e] = (int32_t)(pl.sample_row_off[q] - pl.mb_row_off[j]);
            if (q + 1 == pl.mb_sample_off[j + 1]) a.cu[e + 1] = (int32_t)(pl.sample_row_off[q + 1] - pl.mb_row_off[j]);
          }
        }
        // Is position p inside a placeholder run?  The span table decides (last span with pos_start <= p).
        const uint32_t sbase = slot * v.spans_per_sample, ns = v.s_n_spans[slot];
        uint32_t lo = 0, hi = ns;
        while (lo < hi) {
          const uint32_t mid = (lo + hi) >> 1;
          if (v.sp_pos[sbase + mid] <= p) lo = mid + 1; else hi = mid;
        }
        sid = sbase + lo - 1;
        const bool in_run = lo > 0 && p < v.sp_pos[sid] + v.sp_tokens[sid];
        kind = in_run ? 2 : 1;
        if (!in_run) {
          // token id, through the text page
          const uint64_t tp_gva = v.s_text_pages[(uint64_t)slot * v.text_pages_per_sample + p / kTextPageIds];
          uint64_t off;
          const uint64_t tpte = translate(v, tp_gva, &off);
          text_ok = (tpte & kPteValid) && (tpte & kPteText);  // e.g. a peer's page whose mapping was never imported
          if (text_ok) id = reinterpret_cast<const int32_t*>(tpte & ~kPteFlagMask)[p % kTextPageIds];
        }
      }
      d.out_row = (uint32_t)out_row;
      if (kind == 1) {
        if (!text_ok) {
          note_error(v, a.call_seq, FT_ERR_BAD_GVA, (uint32_t)out_row);
        } else if (id < 0 || (uint32_t)id >= a.vocab) {
          note_error(v, a.call_seq, FT_ERR_BAD_TOKEN_ID, (uint32_t)out_row);
        } else {
          // a table row is one segment in device memory: the low address bits ride in off0
          const uint64_t addr = reinterpret_cast<uint64_t>(a.table + (uint64_t)id * v.row_bytes);
          d.seg[0] = addr & ~kPteFlagMask;
          d.off0 = (uint32_t)(addr & kPteFlagMask);
          d.nseg = 1;
        }
      } else {
        const uint64_t b = (uint64_t)(p - v.sp_pos[sid]) * v.row_bytes;  // byte offset inside the span image
        const uint32_t o0 = (uint32_t)(b >> v.page_shift);
        d.off0 = (uint32_t)(b & (v.page_bytes - 1));
        d.shift = v.page_shift;
        const uint32_t nseg = ((d.off0 + v.row_bytes - 1) >> v.page_shift) + 1;
        bool ok = nseg <= kMaxSeg;
        for (uint32_t s = 0; ok && s < nseg; ++s) {
          uint64_t poff;
          const uint64_t pte = translate(v, span_page_gva(v, sid, o0 + s), &poff);
          ok = (pte & kPteValid) && !(pte & kPteText);
          d.seg[s] = pte;
        }
        if (ok) d.nseg = nseg; else note_error(v, a.call_seq, FT_ERR_BAD_GVA, (uint32_t)out_row);
      }
    }
    desc[buf][lane] = d;
  };

  if (resolver) resolve(0);
  __syncthreads();
  for (uint32_t buf = 0;; buf ^= 1) {
    if (!valid[buf]) break;
    if (resolver) {
      finish_index();    // what the unit just published still owes to cu_seqlens
      resolve(buf ^ 1);  // one unit ahead of the copy
    } else {
      for (uint32_t r = warp; r < R; r += kStreamWarps) {
        const RowDesc& dr = desc[buf][r];
        const uint32_t nseg = dr.nseg;
        if (nseg == 0) continue;
        const uint32_t off0 = dr.off0, shift = dr.shift, mask = (1u << shift) - 1;
        uint4* dst = reinterpret_cast<uint4*>(a.out + (uint64_t)dr.out_row * v.row_bytes);
        auto src_of = [&](uint32_t x, bool* take) -> const uint4* {
          const uint32_t ab = off0 + (x << 4);
          const uint64_t pte = dr.seg[ab >> shift];
          const bool far = (pte & (kPteHost | kPteRemote)) != 0;  // host-tier frame, or a frame in another GPU's HBM
          *take = MODE == kTierAll || !far;                     // (far frames have launches of their own)
          return reinterpret_cast<const uint4*>((pte & ~kPteFlagMask) + (ab & mask));
        };
        // U vectors per lane in flight before the first store
        for (uint32_t x0 = lane; x0 < row_vecs; x0 += 32 * U) {
          uint4 val[U];
          bool take[U];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const uint32_t x = x0 + 32 * u;
            take[u] = false;
            if (x < row_vecs) {
              const uint4* s = src_of(x, &take[u]);
              if (take[u]) val[u] = __ldcs(s);
            }
          }
#pragma unroll
          for (int u = 0; u < U; ++u)
            if (take[u]) __stcs(dst + x0 + 32 * u, val[u]);
        }
      }
    }
    __syncthreads();  // desc[buf ^ 1] is complete, desc[buf] is free
  }
}

// The plan's row words: one thread per output row walks the same tables the resolver's long way walks (plan position,
// span table, text page) and leaves what it found.  Rows whose text page cannot be translated stay unresolved (0).
__global__ void __launch_bounds__(256) k_plan_rows(PoolView v, PlanView pl, uint64_t rows, uint64_t* __restrict__ row_src) {
  for (uint64_t row = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; row < rows; row += (uint64_t)gridDim.x * blockDim.x) {
    uint32_t q = pl.tile_first_sample[row / kTileRows];
    while (row >= pl.sample_row_off[q + 1]) ++q;
    const uint32_t p = (uint32_t)(row - pl.sample_row_off[q]);
    const uint32_t slot = pl.mb_samples[q];
    const uint32_t sbase = slot * v.spans_per_sample, ns = v.s_n_spans[slot];
    uint32_t lo = 0, hi = ns;
    while (lo < hi) {
      const uint32_t mid = (lo + hi) >> 1;
      if (v.sp_pos[sbase + mid] <= p) lo = mid + 1; else hi = mid;
    }
    const uint32_t sid = sbase + lo - 1;
    uint64_t word = 0;
    if (lo > 0 && p < v.sp_pos[sid] + v.sp_tokens[sid]) {
      word = kRowVision | ((uint64_t)p << 32) | sid;
    } else {
      const uint64_t tp_gva = v.s_text_pages[(uint64_t)slot * v.text_pages_per_sample + p / kTextPageIds];
      uint64_t off;
      const uint64_t tpte = translate(v, tp_gva, &off);
      if ((tpte & kPteValid) && (tpte & kPteText)) {
        const int32_t id = reinterpret_cast<const int32_t*>(tpte & ~kPteFlagMask)[p % kTextPageIds];
        word = kRowText | ((uint64_t)p << 32) | (uint32_t)id;
      }
    }
    row_src[row] = word;
  }
}

int32_t plan_rows_launch(ft_pool* p, ft_plan* pl) {
  if (!pl->d_row_src || pl->total_tokens == 0) return FT_OK;
  if (p->have_ids_ev) FT_CUDA(cudaStreamWaitEvent(p->meta, p->ev_ids, 0));  // the ids are a caller's data, copied on its stream
  const uint64_t rows = pl->total_tokens;
  const unsigned grid = (unsigned)std::min<uint64_t>((rows + 255) / 256, (uint64_t)p->sm_count * 16);
  k_plan_rows<<<grid, 256, 0, p->meta>>>(p->view, make_plan_view(pl), rows, pl->d_row_src);
  FT_CUDA(cudaGetLastError());
  ++p->meta_seq;
  ++p->gpu_launches;
  return FT_OK;
}

// Host-tier vision data, page by page.  A span's rows are consecutive output rows, so a page of the span is one
// contiguous byte range of the output: each host-tier page becomes a few bulk copies host frame -> shared ->
// output, read in place over the mapped pointer.  One warp per CTA: the lanes translate 32 page ordinals at a
// time (page list -> GVA -> page-table entry), lane 0 drives the copy ring.  A handful of CTAs saturate the link.
__global__ void __launch_bounds__(32) k_gather_host_bulk(PoolView v, PlanView pl, GatherArgs a, uint64_t want) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint64_t bars[kBulkStages];
  __shared__ uint64_t dst_q[kBulkStages];
  __shared__ uint32_t len_q[kBulkStages];
  const uint32_t lane = threadIdx.x;
  BulkRing ring;
  ring.init(smem, bars, dst_q, len_q, v.bulk_wait_ns, v.bulk_tx_slack);
  uint64_t item = 0;
  // the samples to assemble: the call's range, or the samples of each listed microbatch in turn
  const uint32_t n_parts = a.list ? a.n_list : 1;
  for (uint32_t part = 0; part < n_parts; ++part) {
    uint32_t q_lo = a.q_lo, q_hi = a.q_hi;
    uint64_t part_row_lo = a.row_lo, part_out0 = 0;
    if (a.list) {
      const ListEntry en = a.list[part];
      q_lo = en.q_lo; q_hi = en.q_hi; part_row_lo = en.row_lo; part_out0 = en.out_row0;
    }
    for (uint32_t q = q_lo; q < q_hi; ++q) {
      const uint32_t slot = pl.mb_samples[q], ns = v.s_n_spans[slot];
      uint64_t row0 = part_out0 + (pl.sample_row_off[q] - part_row_lo);
      if (!a.list && a.pad_L) {
        const uint32_t mb = pl.plan_sample_mb[q];
        row0 += (uint64_t)(mb - a.mb_begin) * a.pad_L - (pl.mb_row_off[mb] - a.row_lo);
      }
      for (uint32_t j = 0; j < ns; ++j) {
        const uint32_t sid = slot * v.spans_per_sample + j;
        const uint32_t npages = v.sp_npages[sid];
        const uint64_t nbytes = (uint64_t)v.sp_tokens[sid] * v.row_bytes;
        uint8_t* dst_base = a.out + (row0 + v.sp_pos[sid]) * v.row_bytes;
        for (uint32_t g = 0; g < npages; g += 32, ++item) {
          if (item % gridDim.x != blockIdx.x) continue;
          const uint32_t o = g + lane;
          uint64_t pte = 0, off;
          if (o < npages) pte = translate(v, span_page_gva(v, sid, o), &off);
          const bool mine = (pte & kPteValid) && (pte & want);  // want: kPteHost, or kPteRemote (a peer GPU's HBM)
          const uint32_t mask = __ballot_sync(0xFFFFFFFFu, mine);
          for (uint32_t m = mask; m; m &= m - 1) {
            const int l = __ffs(m) - 1;
            const uint64_t p_l = __shfl_sync(0xFFFFFFFFu, pte, l);
            const uint64_t b0 = (uint64_t)(g + l) << v.page_shift;
            const uint64_t len = min(v.page_bytes, nbytes - b0);
            const uint8_t* src = reinterpret_cast<const uint8_t*>(p_l & ~kPteFlagMask);
            for (uint64_t x = 0; x < len; x += kBulkStageBytes)
              ring.push(src + x, dst_base + b0 + x, (uint32_t)min((uint64_t)kBulkStageBytes, len - x));
          }
        }
      }
    }
  }
  ring.drain();
  if (ring.lost && lane == 0) note_error(v, a.call_seq, FT_ERR_TIMEOUT, (blockIdx.x & 0xFFFFu) | (min(ring.stranded, 0xFFFFu) << 16));
}

}  // namespace ft

namespace ft {
int32_t gather_set_carveout(int pct) {
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierAll, 4, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierAll, 4, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierAll, 8, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierAll, 8, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierDeviceOnly, 4, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierDeviceOnly, 4, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierDeviceOnly, 8, false>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  FT_CUDA(cudaFuncSetAttribute(k_gather<kTierDeviceOnly, 8, true>, cudaFuncAttributePreferredSharedMemoryCarveout, pct));
  return FT_OK;
}
int32_t gather_device_setup(ft_pool* p) {
  FT_CUDA(cudaFuncSetAttribute(k_gather_host_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBulkSmemBytes));
  auto occ = [](auto kernel) { int v = 0; return cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, kernel, kGatherThreads, 0) == cudaSuccess && v > 0 ? v : 1; };
  p->occ_gather[kTierAll][0] = std::min(occ(k_gather<kTierAll, 4, false>), occ(k_gather<kTierAll, 4, true>));
  p->occ_gather[kTierAll][1] = std::min(occ(k_gather<kTierAll, 8, false>), occ(k_gather<kTierAll, 8, true>));
  p->occ_gather[kTierDeviceOnly][0] = std::min(occ(k_gather<kTierDeviceOnly, 4, false>), occ(k_gather<kTierDeviceOnly, 4, true>));
  p->occ_gather[kTierDeviceOnly][1] = std::min(occ(k_gather<kTierDeviceOnly, 8, false>), occ(k_gather<kTierDeviceOnly, 8, true>));
  return FT_OK;
}
}  // namespace ft

namespace ft {
// The launches of one assembly call over microbatches [mb_begin, mb_end): one k_gather, or one per tier.
// pad_L = 0: packed rows, cu_seqlens and position ids written; pad_L = L: rows land in the padded layout and
// the index outputs are left to the caller.  Arguments are validated by the caller.
int32_t gather_launch(ft_pool* p, const ft_plan* pl, uint32_t mb_begin, uint32_t mb_end, const void* embed_table,
                      uint32_t vocab, void* out_embeds, int32_t* out_cu, int32_t* out_pos, uint32_t pad_L, cudaStream_t st,
                      const void* d_list, uint32_t n_list, uint64_t list_tiles, uint64_t list_rows, ClaimCounter* counter,
                      const uint32_t* h_mb_list) {
  if (p->view.row_bytes > (kMaxSeg - 1) * 4096) return FT_ERR_CAPACITY;
  const PlanView pv = make_plan_view(pl);
  const bool listed = d_list != nullptr;
  GatherArgs a;
  a.q_lo = pl->h_mb_sample_off[mb_begin]; a.q_hi = pl->h_mb_sample_off[mb_end]; a.mb_begin = mb_begin;
  a.row_lo = pl->h_mb_row_off[mb_begin]; a.row_hi = pl->h_mb_row_off[mb_end];
  a.table = static_cast<const uint8_t*>(embed_table); a.vocab = vocab;
  a.out = static_cast<uint8_t*>(out_embeds); a.cu = out_cu; a.pos_ids = out_pos;
  a.call_seq = status_seq(p); a.write_index = pad_L == 0; a.pad_L = pad_L;
  a.list = static_cast<const ListEntry*>(d_list); a.n_list = n_list; a.list_tiles = list_tiles;
  const uint64_t n_tiles = listed ? list_tiles : (a.row_hi + kTileRows - 1) / kTileRows - a.row_lo / kTileRows;
  const uint64_t n_rows = listed ? list_rows : a.row_hi - a.row_lo;
  if (n_rows >> 32) return FT_ERR_CAPACITY;  // output row indices are 32-bit inside the kernel
  a.tile_counter = counter;
  // Never more CTAs than fit at once (every CTA claims until the units run out).  Unit size: a range with fewer
  // tiles than CTAs is cut down to 4 rows as long as all units still run in one wave (one resolve, then the copy, per
  // CTA: the latency floor).  Any longer range is cut into units of 8 or 16 rows (one or two rows per copy warp) as
  // long as a unit still streams 48 KiB and more, so that the resolver keeps ahead of the copy: finer units balance
  // the CTAs of an SM and shorten the last wave (6.80 against 6.68 TB/s on a 2.6 M-row range with 7 KiB rows).
  // Launch geometry when the tuning leaves it open: a range of one wave keeps 4 CTAs per SM with 4 vectors per lane
  // in flight (more, smaller units: the latency floor); a longer range of rows of 4 KiB and more streams a little
  // better from 2 CTAs per SM with 8 vectors per lane (the same bytes in flight per SM from half the warps: 6.85
  // against 6.80 TB/s on the long range, 6.26 against 6.15 for one call per microbatch).
  // (Beside a bulk-copy launch for host or remote frames the device-tier launch keeps 4 x 4: 6.70 against 6.57 TB/s.)
  const bool one_launch = !(p->cfg.host_pages != 0 || p->peer_host_frames || p->peer_remote_frames);
  const bool long_range = one_launch && n_tiles > (uint64_t)p->sm_count * 4 && p->view.row_bytes >= 4096;
  const int want_ctas = p->dev_ctas_per_sm ? p->dev_ctas_per_sm : (long_range ? 2 : 4);
  const int unroll = p->gather_unroll ? p->gather_unroll : (long_range ? 8 : 4);
  const uint64_t per_sm_cap = (p->cfg.hbm_pages == 0 && p->cfg.world_size == 1) ? 1 : (uint64_t)want_ctas;
  const uint64_t full_grid = (uint64_t)p->sm_count * per_sm_cap;
  a.sub_shift = 0;
  if (n_tiles <= full_grid) {
    while (a.sub_shift < 3 && (n_tiles << (a.sub_shift + 1)) <= full_grid) ++a.sub_shift;
  } else {
    while (a.sub_shift < 2 && (uint64_t)(kTileRows >> (a.sub_shift + 1)) * p->view.row_bytes >= (48u << 10)) ++a.sub_shift;
  }
  const uint64_t n_units = n_tiles << a.sub_shift;
  auto launch = [&](auto kernel, int mode, uint64_t want_per_sm, const GatherArgs& args, cudaStream_t s) {
    const uint64_t resident = (uint64_t)std::max(1, p->occ_gather[mode][unroll == 8 ? 1 : 0]);
    const uint64_t ctas = (uint64_t)p->sm_count * std::min<uint64_t>(want_per_sm, resident);
    kernel<<<(unsigned)std::min<uint64_t>(n_units, ctas), kGatherThreads, 0, s>>>(p->view, pv, args);
  };
  auto launch_mode = [&](auto mode_tag, const GatherArgs& args, uint64_t want_per_sm) {
    constexpr int M = decltype(mode_tag)::value;
    const bool u8 = unroll == 8;
    if (listed) {
      if (u8) launch(k_gather<M, 8, true>, M, want_per_sm, args, st); else launch(k_gather<M, 4, true>, M, want_per_sm, args, st);
    } else {
      if (u8) launch(k_gather<M, 8, false>, M, want_per_sm, args, st); else launch(k_gather<M, 4, false>, M, want_per_sm, args, st);
    }
  };
  const uint64_t per_sm = per_sm_cap;
  // one launch when only one kind of frame can be a source (own and imported bindings); otherwise one launch per
  // kind: local HBM by vector streams from every SM, host-tier frames and frames in another GPU's HBM each by a
  // few bulk-copy CTAs on a stream of their own (plain bulk copies, each CTA fetching its own bytes)
  const bool host_sources = p->cfg.host_pages != 0 || p->peer_host_frames;
  const bool remote_sources = p->peer_remote_frames;
  const bool only_host = p->cfg.hbm_pages == 0 && !(p->cfg.world_size > 1);
  if ((!host_sources && !remote_sources) || only_host) {
    prof_begin(p, only_host ? FT_K_GATHER_HOST : FT_K_GATHER_DEVICE, st);
    launch_mode(std::integral_constant<int, kTierAll>{}, a, per_sm);
    prof_end(p, st);
    p->gpu_launches += 1;
  } else {
    GatherArgs ah = a;
    ah.write_index = 0;
    if (host_sources) {
      FT_CUDA(cudaEventRecord(p->fork_ev[1], st));
      FT_CUDA(cudaStreamWaitEvent(p->side_stream[1], p->fork_ev[1], 0));
      prof_begin(p, FT_K_GATHER_HOST, p->side_stream[1]);
      if (host_tier_by_copy_engine(p) && pl->host_copies_valid && !p->peer_host_frames && (!listed || h_mb_list)) {
        // the host tier through the copy engine: every run of host pages of the microbatches asked for is one
        // contiguous byte range of the output (a span's rows are consecutive output rows)
        const uint64_t rb = p->view.row_bytes;
        auto issue = [&](uint32_t j, uint64_t out_row0) -> int32_t {  // out_row0: output row of the microbatch's first row
          for (uint32_t e = pl->mb_copy_off[j]; e < pl->mb_copy_off[j + 1]; ++e) {
            const ft_plan::HostCopy& hc = pl->host_copies[e];
            uint8_t* dst = a.out + (out_row0 + (hc.row0 - pl->h_mb_row_off[j])) * rb + hc.img_off;
            FT_CUDA(cudaMemcpyAsync(dst, hc.src, hc.len, cudaMemcpyHostToDevice, p->side_stream[1]));
          }
          return FT_OK;
        };
        uint64_t out_row0 = 0;
        if (listed) {
          for (uint32_t i = 0; i < n_list; ++i) {
            const uint32_t j = h_mb_list[i];
            const int32_t rcj = issue(j, out_row0);
            if (rcj != FT_OK) return rcj;
            out_row0 += pl->h_mb_row_off[j + 1] - pl->h_mb_row_off[j];
          }
        } else {
          for (uint32_t j = mb_begin; j < mb_end; ++j) {
            const int32_t rcj = issue(j, pad_L ? (uint64_t)(j - mb_begin) * pad_L : pl->h_mb_row_off[j] - a.row_lo);
            if (rcj != FT_OK) return rcj;
          }
        }
      } else {
        k_gather_host_bulk<<<(unsigned)p->host_ctas, 32, kBulkSmemBytes, p->side_stream[1]>>>(p->view, pv, ah, kPteHost);
        p->gpu_launches += 1;
      }
      prof_end(p, p->side_stream[1]);
      FT_CUDA(cudaEventRecord(p->join_ev[1], p->side_stream[1]));
    }
    if (remote_sources) {
      FT_CUDA(cudaEventRecord(p->fork_ev[2], st));
      FT_CUDA(cudaStreamWaitEvent(p->side_stream[2], p->fork_ev[2], 0));
      prof_begin(p, FT_K_GATHER_REMOTE, p->side_stream[2]);
      k_gather_host_bulk<<<(unsigned)p->remote_ctas, 32, kBulkSmemBytes, p->side_stream[2]>>>(p->view, pv, ah, kPteRemote);
      prof_end(p, p->side_stream[2]);
      FT_CUDA(cudaEventRecord(p->join_ev[2], p->side_stream[2]));
      p->gpu_launches += 1;
    }
    prof_begin(p, FT_K_GATHER_DEVICE, st);
    launch_mode(std::integral_constant<int, kTierDeviceOnly>{}, a, per_sm);
    prof_end(p, st);
    if (host_sources) FT_CUDA(cudaStreamWaitEvent(st, p->join_ev[1], 0));
    if (remote_sources) FT_CUDA(cudaStreamWaitEvent(st, p->join_ev[2], 0));
    p->gpu_launches += 1;
  }
  FT_CUDA(cudaGetLastError());
  p->bytes_gathered += n_rows * 2ull * p->view.row_bytes;
  return FT_OK;
}
}  // namespace ft

using namespace ft;

extern "C" __attribute__((visibility("default"))) int32_t pool_gather_packed(ft_pool* p, const ft_plan* pl, uint32_t mb_begin, uint32_t mb_end,
                                      const void* embed_table, uint32_t vocab, void* out_embeds, int32_t* out_cu,
                                      int32_t* out_pos, void* stream) {
  if (!p || !pl || pl->pool != p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (mb_begin > mb_end || mb_end > pl->n_mb) return FT_ERR_INVALID_ARG;
  {
    const int32_t alive = plan_alive(p, pl);
    if (alive != FT_OK) return alive;
  }
  if (mb_begin == mb_end) return FT_OK;
  if (!embed_table || !out_embeds || !out_cu || !out_pos) return FT_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(out_embeds) & 15 || reinterpret_cast<uintptr_t>(embed_table) & 15) return FT_ERR_INVALID_ARG;
  if (p->view.row_bytes > (kMaxSeg - 1) * 4096) return FT_ERR_CAPACITY;

  {
    const int32_t rc0 = begin_consumer(p, static_cast<cudaStream_t>(stream));  // writes issued on another stream come first
    if (rc0 != FT_OK) return rc0;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ft_call_ctx* cx = nullptr;
  {
    const int32_t rc1 = ctx_acquire(p, 1, 0, 0, &cx, false, st);  // for its claim counter
    if (rc1 != FT_OK) return rc1;
  }
  {
    const int32_t rc1 = gather_launch(p, pl, mb_begin, mb_end, embed_table, vocab, out_embeds, out_cu, out_pos, 0, st, nullptr, 0, 0, 0, cx->counters);
    if (rc1 != FT_OK) return rc1;
  }
  {
    const int32_t rc1 = ctx_release(p, cx, st);
    if (rc1 != FT_OK) return rc1;
  }
  const_cast<ft_plan*>(pl)->last_stream = st;
  return end_consumer(p, st);
}

extern "C" __attribute__((visibility("default"))) int32_t pool_gather_list(ft_pool* p, const ft_plan* pl, const uint32_t* mb_list, uint32_t n_list,
                                                                           const void* embed_table, uint32_t vocab, void* out_embeds, int32_t* out_cu,
                                                                           int32_t* out_pos, void* stream) {
  if (!p || !pl || pl->pool != p || (n_list && !mb_list)) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  for (uint32_t i = 0; i < n_list; ++i)
    if (mb_list[i] >= pl->n_mb) return FT_ERR_INVALID_ARG;
  {
    const int32_t alive = plan_alive(p, pl);
    if (alive != FT_OK) return alive;
  }
  if (n_list == 0) return FT_OK;
  if (!embed_table || !out_embeds || !out_cu || !out_pos) return FT_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(out_embeds) & 15 || reinterpret_cast<uintptr_t>(embed_table) & 15) return FT_ERR_INVALID_ARG;
  if (p->view.row_bytes > (kMaxSeg - 1) * 4096) return FT_ERR_CAPACITY;
  // one entry per listed microbatch: its plan rows, and where its tiles, output rows and cu_seqlens entries start
  std::vector<ListEntry> entries(n_list);
  uint64_t tiles = 0, rows = 0, cu = 0;
  for (uint32_t i = 0; i < n_list; ++i) {
    const uint32_t j = mb_list[i];
    ListEntry& en = entries[i];
    en.row_lo = pl->h_mb_row_off[j]; en.row_hi = pl->h_mb_row_off[j + 1];
    en.q_lo = pl->h_mb_sample_off[j]; en.q_hi = pl->h_mb_sample_off[j + 1];
    en.tile0 = tiles; en.out_row0 = rows; en.cu0 = (uint32_t)cu; en.pad = 0;
    tiles += (en.row_hi + kTileRows - 1) / kTileRows - en.row_lo / kTileRows;
    rows += en.row_hi - en.row_lo;
    cu += (uint64_t)(en.q_hi - en.q_lo) + 1;
  }
  if ((rows >> 32) || (cu >> 32)) return FT_ERR_CAPACITY;  // output row indices are 32-bit inside the kernels
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = entries.size() * sizeof(ListEntry);
  ft_call_ctx* cx = nullptr;
  {
    int32_t rc1 = ctx_acquire(p, 1, bytes, bytes, &cx);
    if (rc1 != FT_OK) return rc1;
    memcpy(cx->h, entries.data(), bytes);
    if ((rc1 = ctx_upload(p, cx, bytes)) != FT_OK) return rc1;  // on the metadata stream; begin_consumer orders `st` behind it
  }
  {
    const int32_t rc0 = begin_consumer(p, st);
    if (rc0 != FT_OK) return rc0;
  }
  {
    const int32_t rc2 = gather_launch(p, pl, 0, pl->n_mb, embed_table, vocab, out_embeds, out_cu, out_pos, 0, st, cx->d, n_list, tiles, rows, cx->counters, mb_list);
    if (rc2 != FT_OK) return rc2;
  }
  {
    const int32_t rc3 = ctx_release(p, cx, st);
    if (rc3 != FT_OK) return rc3;
  }
  const_cast<ft_plan*>(pl)->last_stream = st;
  return end_consumer(p, st);
}
