// Backbone-side outputs next to assembly: the padded layout (every microbatch occupies exactly L rows),
// three-component positions, token ids, next-token labels and loss mask, and the gradient of the embedding
// table through the assembled input.  The paper stops at "the backbone consumes microbatches" (Sec. 3.1);
// these are the library's own definitions, stated in the public header.  What the paper fixes and this file
// relies on: image and text subsequences are interleaved (Sec. 4.1), a microbatch holds at most L tokens
// (Sec. 3.4), and the encoders are frozen, so no gradient flows back into the pool's pages.
//
//   k_set_grids      stores the (T, H, W) token grids of named spans
//   k_pad_zero       zero rows behind the last token of each microbatch (16-byte streaming stores)
//   k_backbone_index one thread per padded row: cu_seqlens, positions, ids, labels, mask
//   k_grad_row_ids   one thread per row of the gradient's layout: the table row it adds to, or -1
//   k_embed_grad     one CTA per range of table rows: walks the row ids in ascending order and adds the rows
//                    that fall in its range, so every table element sees its additions in row order
#include <algorithm>
#include <vector>

#include "flowpool_internal.cuh"

namespace ft {

constexpr int32_t kIgnoreLabel = -100;

struct GridCall {
  uint32_t n;
  const uint32_t* span_id;  // slot * spans_per_sample + span index
  const uint4* grid;
};

__global__ void k_set_grids(PoolView v, GridCall c) {
  const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < c.n) v.sp_grid[c.span_id[i]] = c.grid[i];
}

// A row of a layout -> (plan position q, position p inside the sample).  Packed layout: rows of the range are
// consecutive; padded layout: microbatch j of the range starts at row (j - mb_begin) * L.
struct RowAt {
  uint32_t q, p, slot, seq_len, mb;
  bool real;  // false: a padding row
};

struct LayoutArgs {
  uint32_t mb_begin, mb_end, q_lo, q_hi, L;
  uint32_t padded;
  uint64_t row_lo;  // plan-global packed row of the range's first row
  uint64_t rows;    // rows of the layout
};

__device__ __forceinline__ RowAt row_at(const PlanView& pl, const LayoutArgs& a, uint64_t R) {
  RowAt r;
  r.real = false; r.q = 0; r.p = 0; r.slot = 0; r.seq_len = 0;
  uint64_t row;
  uint32_t lo, hi;
  if (a.padded) {
    r.mb = a.mb_begin + (uint32_t)(R / a.L);
    const uint64_t t = R % a.L;
    if (t >= pl.mb_row_off[r.mb + 1] - pl.mb_row_off[r.mb]) return r;
    row = pl.mb_row_off[r.mb] + t;
    lo = pl.mb_sample_off[r.mb]; hi = pl.mb_sample_off[r.mb + 1];
  } else {
    row = a.row_lo + R;
    lo = a.q_lo; hi = a.q_hi;
  }
  // last plan position whose first row is <= row
  while (hi - lo > 1) {
    const uint32_t mid = (lo + hi) >> 1;
    if (pl.sample_row_off[mid] <= row) lo = mid; else hi = mid;
  }
  r.q = lo;
  r.p = (uint32_t)(row - pl.sample_row_off[lo]);
  r.seq_len = (uint32_t)(pl.sample_row_off[lo + 1] - pl.sample_row_off[lo]);
  r.slot = pl.mb_samples[lo];
  if (!a.padded) r.mb = pl.plan_sample_mb[lo];
  r.real = true;
  return r;
}

// index of the span whose run holds position p, or kNone
__device__ __forceinline__ uint32_t span_holding(const PoolView& v, uint32_t slot, uint32_t p) {
  const uint32_t sbase = slot * v.spans_per_sample, ns = v.s_n_spans[slot];
  uint32_t lo = 0, hi = ns;
  while (lo < hi) {
    const uint32_t mid = (lo + hi) >> 1;
    if (v.sp_pos[sbase + mid] <= p) lo = mid + 1; else hi = mid;
  }
  if (lo == 0) return kNone;
  const uint32_t sid = sbase + lo - 1;
  return p < v.sp_pos[sid] + v.sp_tokens[sid] ? sid : kNone;
}

// token id at position p of a slot, through the text page; false when the text page does not translate
__device__ __forceinline__ bool token_id_at(const PoolView& v, uint32_t slot, uint32_t p, int32_t* id) {
  const uint64_t tp_gva = v.s_text_pages[(uint64_t)slot * v.text_pages_per_sample + p / kTextPageIds];
  uint64_t off;
  const uint64_t tpte = translate(v, tp_gva, &off);
  if (!((tpte & kPteValid) && (tpte & kPteText))) return false;
  *id = reinterpret_cast<const int32_t*>(tpte & ~kPteFlagMask)[p % kTextPageIds];
  return true;
}

struct IndexArgs {
  LayoutArgs lay;
  int32_t pad_id;
  int32_t *cu, *pos3, *ids, *labels;
  uint8_t* mask;
  uint64_t call_seq;
};

__global__ void __launch_bounds__(256) k_backbone_index(PoolView v, PlanView pl, IndexArgs a) {
  const uint64_t R = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (R >= a.lay.rows) return;
  const RowAt r = row_at(pl, a.lay, R);
  const uint32_t t = (uint32_t)(R % a.lay.L);
  // cu_seqlens of microbatch j: 0, the sample ends, then L (the padding as one last sequence)
  const uint64_t e_base = (uint64_t)(pl.mb_sample_off[r.mb] - a.lay.q_lo) + 2ull * (r.mb - a.lay.mb_begin);
  if (t == 0) {
    a.cu[e_base] = 0;
    a.cu[e_base + (pl.mb_sample_off[r.mb + 1] - pl.mb_sample_off[r.mb]) + 1] = (int32_t)a.lay.L;
  }
  if (!r.real) {
    a.pos3[R] = 0; a.pos3[a.lay.rows + R] = 0; a.pos3[2 * a.lay.rows + R] = 0;
    a.ids[R] = a.pad_id; a.labels[R] = kIgnoreLabel; a.mask[R] = 0;
    return;
  }
  if (r.p == 0)
    a.cu[e_base + (r.q - pl.mb_sample_off[r.mb]) + 1] = (int32_t)(pl.sample_row_off[r.q + 1] - pl.mb_row_off[r.mb]);
  int32_t id = -1, next_id = -1;
  bool ok = token_id_at(v, r.slot, r.p, &id);
  bool has_label = false;
  if (r.p + 1 < r.seq_len && span_holding(v, r.slot, r.p + 1) == kNone) {
    ok = token_id_at(v, r.slot, r.p + 1, &next_id) && ok;
    has_label = true;
  }
  if (!ok) note_error(v, a.call_seq, FT_ERR_BAD_GVA, (uint32_t)R);
  a.ids[R] = id;
  a.labels[R] = has_label ? next_id : kIgnoreLabel;
  a.mask[R] = has_label ? 1 : 0;
  // Three-component position: a counter st runs over the sample; a text token (or a token of a span without a
  // grid) takes (st, st, st) and advances st by 1; a span with grid (T, H, W) that starts at counter st gives its
  // token (t, h, w) the position (st + t, st + h, st + w) and advances st by max(T, H, W).  So st at position p is
  // p minus, for every gridded span that ends at or before p, (tokens - largest extent).
  const uint32_t sbase = r.slot * v.spans_per_sample, ns = v.s_n_spans[r.slot];
  uint32_t shrink = 0;
  int32_t c0, c1, c2;
  bool in_grid = false;
  for (uint32_t k = 0; k < ns; ++k) {
    const uint32_t ps = v.sp_pos[sbase + k], n = v.sp_tokens[sbase + k];
    if (ps > r.p) break;
    const uint4 g = v.sp_grid[sbase + k];
    if (r.p < ps + n) {
      if (g.x) {
        const uint32_t i = r.p - ps, base = ps - shrink;
        c0 = (int32_t)(base + i / (g.y * g.z)); c1 = (int32_t)(base + (i / g.z) % g.y); c2 = (int32_t)(base + i % g.z);
        in_grid = true;
      }
      break;
    }
    if (g.x) shrink += n - max(g.x, max(g.y, g.z));
  }
  if (!in_grid) c0 = c1 = c2 = (int32_t)(r.p - shrink);
  a.pos3[R] = c0; a.pos3[a.lay.rows + R] = c1; a.pos3[2 * a.lay.rows + R] = c2;
}

// Zero rows behind the last token of each microbatch of the range.  The padding of all microbatches, cut into
// 64 KiB chunks, is dealt round-robin over the CTAs of a grid that fills the device once, so one nearly empty
// microbatch (the last of a plan) is zeroed by the whole grid, not by a few CTAs.
constexpr uint32_t kPadChunkVecs = 4096;  // 16-byte vectors per chunk
__global__ void __launch_bounds__(256) k_pad_zero(PlanView pl, LayoutArgs a, uint32_t row_bytes, uint8_t* out) {
  const uint4 z = make_uint4(0, 0, 0, 0);
  uint64_t base = 0;  // chunks of the microbatches before j
  for (uint32_t j = a.mb_begin; j < a.mb_end; ++j) {
    const uint64_t tokens = pl.mb_row_off[j + 1] - pl.mb_row_off[j];
    const uint64_t vecs = (a.L - tokens) * (uint64_t)(row_bytes >> 4);
    const uint64_t chunks = (vecs + kPadChunkVecs - 1) / kPadChunkVecs;
    uint4* dst = reinterpret_cast<uint4*>(out + ((uint64_t)(j - a.mb_begin) * a.L + tokens) * row_bytes);
    // this CTA's chunks of microbatch j: global chunk index base + k congruent to blockIdx.x modulo the grid
    uint64_t k = (blockIdx.x + gridDim.x - base % gridDim.x) % gridDim.x;
    for (; k < chunks; k += gridDim.x) {
      const uint64_t x0 = k * kPadChunkVecs, x1 = min(vecs, x0 + kPadChunkVecs);
      for (uint64_t x = x0 + threadIdx.x; x < x1; x += blockDim.x) __stcs(dst + x, z);
    }
    base += chunks;
  }
}

}  // namespace ft

namespace ft {

struct RowIdArgs {
  LayoutArgs lay;
  uint32_t vocab;
  int32_t* row_id;
  uint64_t call_seq;
};

// The table row each row of the gradient's layout adds to: its token id at a text position, -1 at a span
// position (frozen encoders: nothing flows back into the pool) and on padding.
__global__ void __launch_bounds__(256) k_grad_row_ids(PoolView v, PlanView pl, RowIdArgs a) {
  const uint64_t R = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (R >= a.lay.rows) return;
  int32_t out = -1;
  const RowAt r = row_at(pl, a.lay, R);
  if (r.real && span_holding(v, r.slot, r.p) == kNone) {
    int32_t id = -1;
    if (!token_id_at(v, r.slot, r.p, &id)) note_error(v, a.call_seq, FT_ERR_BAD_GVA, (uint32_t)R);
    else if (id < 0 || (uint32_t)id >= a.vocab) note_error(v, a.call_seq, FT_ERR_BAD_TOKEN_ID, (uint32_t)R);
    else out = id;
  }
  a.row_id[R] = out;
}

constexpr int kGradThreads = 256;
constexpr uint32_t kGradChunk = 4 * kGradThreads;  // row ids examined per round: four per thread

__device__ __forceinline__ int4 load_ids4(const int32_t* row_id, uint64_t r0, uint64_t rows) {
  if (r0 + 3 < rows) return *reinterpret_cast<const int4*>(row_id + r0);
  int4 x = make_int4(-1, -1, -1, -1);
  if (r0 < rows) x.x = row_id[r0];
  if (r0 + 1 < rows) x.y = row_id[r0 + 1];
  if (r0 + 2 < rows) x.z = row_id[r0 + 2];
  return x;
}

// CTA b owns the table rows v with v % gridDim.x == b.  It walks all row ids in ascending row order, a chunk at
// a time, keeps the rows it owns (order-preserving compaction: four consecutive rows per thread, warp scan,
// warp totals), and adds them one row after the other, each thread always on the same columns: every table
// element receives its additions in ascending row order, one rounded fp32 addition each, whatever the grid.
__global__ void __launch_bounds__(kGradThreads) k_embed_grad(const int32_t* __restrict__ row_id, uint64_t rows, uint32_t H,
                                                             const uint4* __restrict__ grad, float* table) {
  __shared__ uint32_t s_row[kGradChunk];
  __shared__ int32_t s_id[kGradChunk];
  __shared__ uint32_t s_warp[kGradThreads / 32];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t vec_per_row = H >> 3;
  int4 cur = load_ids4(row_id, 4ull * threadIdx.x, rows);
  for (uint64_t base = 0; base < rows; base += kGradChunk) {
    const int4 nxt = load_ids4(row_id, base + kGradChunk + 4ull * threadIdx.x, rows);  // in flight while this chunk is added
    const int32_t ids[4] = {cur.x, cur.y, cur.z, cur.w};
    uint32_t mine = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) mine |= (ids[k] >= 0 && (uint32_t)ids[k] % gridDim.x == blockIdx.x) ? 1u << k : 0u;
    const uint32_t cnt = __popc(mine);
    uint32_t incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
      if (lane >= d) incl += up;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    uint32_t off = incl - cnt, total = 0;
#pragma unroll
    for (int w2 = 0; w2 < kGradThreads / 32; ++w2) {
      const uint32_t c = s_warp[w2];
      if (w2 < (int)warp) off += c;
      total += c;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (mine & (1u << k)) { s_row[off] = 4 * threadIdx.x + k; s_id[off] = ids[k]; ++off; }
    __syncthreads();
    for (uint32_t e = 0; e < total; ++e) {
      const uint4* g = grad + (base + s_row[e]) * vec_per_row;
      float4* t = reinterpret_cast<float4*>(table + (uint64_t)s_id[e] * H);
      for (uint32_t x = threadIdx.x; x < vec_per_row; x += kGradThreads) {
        const uint4 gv = __ldcs(g + x);  // eight bf16 values; widening to fp32 is exact
        float4 a = t[2 * x], b = t[2 * x + 1];
        a.x = __fadd_rn(a.x, __uint_as_float(gv.x << 16)); a.y = __fadd_rn(a.y, __uint_as_float(gv.x & 0xFFFF0000u));
        a.z = __fadd_rn(a.z, __uint_as_float(gv.y << 16)); a.w = __fadd_rn(a.w, __uint_as_float(gv.y & 0xFFFF0000u));
        b.x = __fadd_rn(b.x, __uint_as_float(gv.z << 16)); b.y = __fadd_rn(b.y, __uint_as_float(gv.z & 0xFFFF0000u));
        b.z = __fadd_rn(b.z, __uint_as_float(gv.w << 16)); b.w = __fadd_rn(b.w, __uint_as_float(gv.w & 0xFFFF0000u));
        t[2 * x] = a; t[2 * x + 1] = b;
      }
    }
    __syncthreads();  // the lists are rewritten next round
    cur = nxt;
  }
}

// a plan dies with any of its samples (freed, or never completed under ALLOW_UNWRITTEN)
static int32_t plan_alive(const ft_pool* p, const ft_plan* pl) {
  if (pl->free_epoch != p->free_epoch || (pl->cfg.flags & FT_PLAN_ALLOW_UNWRITTEN)) {
    for (uint32_t t = 0; t < pl->n; ++t) {
      const ft_slot_mirror& s = p->slots[pl->slots[t]];
      if (s.state != FT_SLOT_READY || s.generation != pl->slot_generation[t]) return FT_ERR_NOT_READY;
    }
  }
  return FT_OK;
}

static LayoutArgs layout_of(const ft_plan* pl, uint32_t mb_begin, uint32_t mb_end, bool padded) {
  LayoutArgs a;
  a.mb_begin = mb_begin; a.mb_end = mb_end;
  a.q_lo = pl->h_mb_sample_off[mb_begin]; a.q_hi = pl->h_mb_sample_off[mb_end];
  a.L = pl->cfg.budget_L; a.padded = padded ? 1 : 0;
  a.row_lo = pl->h_mb_row_off[mb_begin];
  a.rows = padded ? (uint64_t)(mb_end - mb_begin) * a.L : pl->h_mb_row_off[mb_end] - pl->h_mb_row_off[mb_begin];
  return a;
}

}  // namespace ft

using namespace ft;

extern "C" __attribute__((visibility("default"))) int32_t pool_set_span_grids(ft_pool* p, uint32_t n, const uint32_t* slot, const uint32_t* span_idx,
                                                                              const uint32_t* grid_thw, void* stream) {
  if (!p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (n == 0) return FT_OK;
  if (!slot || !span_idx || !grid_thw) return FT_ERR_INVALID_ARG;
  const uint32_t S = p->cfg.max_spans_per_sample;
  for (uint32_t i = 0; i < n; ++i) {
    if (slot[i] >= p->cfg.max_samples) return FT_ERR_INVALID_ARG;
    const ft_slot_mirror& s = p->slots[slot[i]];
    if (s.state == FT_SLOT_FREE) return FT_ERR_UNKNOWN_SAMPLE;
    if (span_idx[i] >= s.n_spans) return FT_ERR_INVALID_ARG;
    const uint32_t* g = grid_thw + 3ull * i;
    if (g[0] == 0 || g[1] == 0 || g[2] == 0) return FT_ERR_INVALID_ARG;
    // T*H*W == tokens without overflow: the running product never exceeds the (32-bit) token count
    const uint64_t tokens = p->spans[(size_t)slot[i] * S + span_idx[i]].tokens;
    const uint64_t th = (uint64_t)g[0] * g[1];
    if (th > tokens || th * g[2] != tokens) return FT_ERR_INVALID_ARG;
  }
  const size_t o_grid = 0, o_sid = align_up_sz((size_t)n * sizeof(uint4), 16), bytes = o_sid + (size_t)n * 4;
  std::vector<uint8_t> blob(bytes);
  uint4* hg = reinterpret_cast<uint4*>(blob.data() + o_grid);
  uint32_t* hs = reinterpret_cast<uint32_t*>(blob.data() + o_sid);
  for (uint32_t i = 0; i < n; ++i) {
    hg[i] = make_uint4(grid_thw[3ull * i], grid_thw[3ull * i + 1], grid_thw[3ull * i + 2], 0);
    hs[i] = slot[i] * S + span_idx[i];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    const int32_t rc0 = begin_free(p, st);  // assemblies issued on another stream read the grids first
    if (rc0 != FT_OK) return rc0;
  }
  void* d = nullptr;
  const int32_t rc = stage_upload(p, 0, blob.data(), bytes, bytes, st, &d);
  if (rc != FT_OK) return rc;
  GridCall c;
  c.n = n;
  c.grid = reinterpret_cast<const uint4*>(static_cast<uint8_t*>(d) + o_grid);
  c.span_id = reinterpret_cast<const uint32_t*>(static_cast<uint8_t*>(d) + o_sid);
  k_set_grids<<<(n + 255) / 256, 256, 0, st>>>(p->view, c);
  FT_CUDA(cudaGetLastError());
  p->gpu_launches += 1;
  return end_producer(p, st);
}

extern "C" __attribute__((visibility("default"))) int32_t pool_gather_padded(ft_pool* p, const ft_plan* pl, uint32_t mb_begin, uint32_t mb_end,
                                                                             const void* embed_table, uint32_t vocab, int32_t pad_id, void* out_embeds,
                                                                             int32_t* out_cu, int32_t* out_pos3, int32_t* out_ids, int32_t* out_labels,
                                                                             uint8_t* out_mask, void* stream) {
  if (!p || !pl || pl->pool != p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (mb_begin > mb_end || mb_end > pl->n_mb) return FT_ERR_INVALID_ARG;
  {
    const int32_t rc0 = plan_alive(p, pl);
    if (rc0 != FT_OK) return rc0;
  }
  if (mb_begin == mb_end) return FT_OK;
  if (!embed_table || !out_embeds || !out_cu || !out_pos3 || !out_ids || !out_labels || !out_mask) return FT_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(out_embeds) & 15 || reinterpret_cast<uintptr_t>(embed_table) & 15) return FT_ERR_INVALID_ARG;
  const LayoutArgs lay = layout_of(pl, mb_begin, mb_end, true);
  if (lay.rows >> 32) return FT_ERR_CAPACITY;  // padded row indices are 32-bit inside the kernels
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    const int32_t rc0 = begin_consumer(p, st);
    if (rc0 != FT_OK) return rc0;
  }
  {
    const int32_t rc1 = gather_launch(p, pl, mb_begin, mb_end, embed_table, vocab, out_embeds, nullptr, nullptr, lay.L, st);
    if (rc1 != FT_OK) return rc1;
  }
  const PlanView pv = make_plan_view(pl);
  k_pad_zero<<<(unsigned)p->sm_count * 8, 256, 0, st>>>(pv, lay, p->view.row_bytes, static_cast<uint8_t*>(out_embeds));
  IndexArgs ia;
  ia.lay = lay; ia.pad_id = pad_id; ia.cu = out_cu; ia.pos3 = out_pos3; ia.ids = out_ids; ia.labels = out_labels;
  ia.mask = out_mask; ia.call_seq = p->call_seq;
  k_backbone_index<<<(unsigned)((lay.rows + 255) / 256), 256, 0, st>>>(p->view, pv, ia);
  FT_CUDA(cudaGetLastError());
  p->gpu_launches += 2;
  const_cast<ft_plan*>(pl)->last_stream = st;
  return end_consumer(p, st);
}

extern "C" __attribute__((visibility("default"))) int32_t pool_embed_grad(ft_pool* p, const ft_plan* pl, uint32_t mb_begin, uint32_t mb_end,
                                                                          uint32_t padded, const void* grad_out, float* grad_table, uint32_t vocab,
                                                                          void* stream) {
  if (!p || !pl || pl->pool != p) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  if (mb_begin > mb_end || mb_end > pl->n_mb) return FT_ERR_INVALID_ARG;
  {
    const int32_t rc0 = plan_alive(p, pl);
    if (rc0 != FT_OK) return rc0;
  }
  if (mb_begin == mb_end) return FT_OK;
  if (!grad_out || !grad_table || vocab == 0) return FT_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(grad_out) & 15 || reinterpret_cast<uintptr_t>(grad_table) & 15) return FT_ERR_INVALID_ARG;
  const LayoutArgs lay = layout_of(pl, mb_begin, mb_end, padded != 0);
  if (lay.rows == 0) return FT_OK;
  if (lay.rows >> 32) return FT_ERR_CAPACITY;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    const int32_t rc0 = begin_consumer(p, st);
    if (rc0 != FT_OK) return rc0;
  }
  int32_t* row_id = nullptr;
  FT_CUDA(cudaMallocAsync(reinterpret_cast<void**>(&row_id), (lay.rows + 4) * 4, st));
  RowIdArgs ra;
  ra.lay = lay; ra.vocab = vocab; ra.row_id = row_id; ra.call_seq = p->call_seq;
  const PlanView pv = make_plan_view(pl);
  k_grad_row_ids<<<(unsigned)((lay.rows + 255) / 256), 256, 0, st>>>(p->view, pv, ra);
  const uint32_t ctas = std::min<uint32_t>(vocab, (uint32_t)p->sm_count * (uint32_t)p->grad_ctas_per_sm);
  prof_begin(p, FT_K_EMBED_GRAD, st);
  k_embed_grad<<<ctas, kGradThreads, 0, st>>>(row_id, lay.rows, p->view.hidden, static_cast<const uint4*>(grad_out), grad_table);
  prof_end(p, st);
  const cudaError_t e = cudaGetLastError();
  cudaFreeAsync(row_id, st);
  if (e != cudaSuccess) return cuda_fail(e, "k_embed_grad");
  p->gpu_launches += 2;
  const_cast<ft_plan*>(pl)->last_stream = st;
  return end_consumer(p, st);
}
