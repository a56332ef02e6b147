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
//   k_embed_grad     CTA b owns the table rows v % grid == b: walks the list of the rest in ascending row order
//                    and adds the rows it owns, so every table element sees its additions in row order
//   k_hot_select     ids with many rows
//   k_split_count / k_split_scan / k_split_fill   stable split of the adding rows: one list per frequent id,
//                    one list (row, id) for the rest
//   k_embed_grad_hot one CTA per (frequent id, 256-column slice): streams the listed rows, adds in list order
#include <algorithm>
#include <cstring>
#include <unordered_set>
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
  uint32_t* id_count;  // [vocab], zero at launch: rows per table row
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
    else { out = id; atomicAdd(a.id_count + id, 1u); }
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

// eight bf16 values added to eight fp32 accumulators; widening bf16 to fp32 is exact, each addition rounds once
__device__ __forceinline__ void add8(float4& a, float4& b, const uint4 gv) {
  a.x = __fadd_rn(a.x, __uint_as_float(gv.x << 16)); a.y = __fadd_rn(a.y, __uint_as_float(gv.x & 0xFFFF0000u));
  a.z = __fadd_rn(a.z, __uint_as_float(gv.y << 16)); a.w = __fadd_rn(a.w, __uint_as_float(gv.y & 0xFFFF0000u));
  b.x = __fadd_rn(b.x, __uint_as_float(gv.z << 16)); b.y = __fadd_rn(b.y, __uint_as_float(gv.z & 0xFFFF0000u));
  b.z = __fadd_rn(b.z, __uint_as_float(gv.w << 16)); b.w = __fadd_rn(b.w, __uint_as_float(gv.w & 0xFFFF0000u));
}

__device__ __forceinline__ uint4 load_rows4(const uint32_t* rows, uint64_t r0, uint64_t n) {
  if (r0 + 3 < n) return *reinterpret_cast<const uint4*>(rows + r0);
  uint4 x = make_uint4(0, 0, 0, 0);
  if (r0 < n) x.x = rows[r0];
  if (r0 + 1 < n) x.y = rows[r0 + 1];
  if (r0 + 2 < n) x.z = rows[r0 + 2];
  return x;
}

// CTA b owns the table rows v with v % gridDim.x == b.  It walks the list of adding rows (ascending; rows of
// frequent ids, span rows and padding are not in it), a chunk at a time, keeps the entries it owns
// (order-preserving compaction: four consecutive entries per thread, warp scan, warp totals), and adds them one
// row after the other, each thread always on the same columns: every table element receives its additions in
// ascending row order, one rounded fp32 addition each, whatever the grid.
__global__ void __launch_bounds__(kGradThreads) k_embed_grad(const int32_t* __restrict__ list_id, const uint32_t* __restrict__ list_row,
                                                             const uint32_t* __restrict__ n_list, uint32_t H,
                                                             const uint4* __restrict__ grad, float* table) {
  __shared__ uint32_t s_row[kGradChunk];
  __shared__ int32_t s_id[kGradChunk];
  __shared__ uint32_t s_warp[kGradThreads / 32];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t vec_per_row = H >> 3;
  const uint64_t n = *n_list;
  int4 cur = load_ids4(list_id, 4ull * threadIdx.x, n);
  uint4 cur_r = load_rows4(list_row, 4ull * threadIdx.x, n);
  for (uint64_t base = 0; base < n; base += kGradChunk) {
    // the next chunk is in flight while this one is added
    const int4 nxt = load_ids4(list_id, base + kGradChunk + 4ull * threadIdx.x, n);
    const uint4 nxt_r = load_rows4(list_row, base + kGradChunk + 4ull * threadIdx.x, n);
    const int32_t ids[4] = {cur.x, cur.y, cur.z, cur.w};
    const uint32_t rws[4] = {cur_r.x, cur_r.y, cur_r.z, cur_r.w};
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
      if (mine & (1u << k)) { s_row[off] = rws[k]; s_id[off] = ids[k]; ++off; }
    __syncthreads();
    for (uint32_t e = 0; e < total; ++e) {
      const uint4* g = grad + (uint64_t)s_row[e] * vec_per_row;
      float4* t = reinterpret_cast<float4*>(table + (uint64_t)s_id[e] * H);
      for (uint32_t x = threadIdx.x; x < vec_per_row; x += kGradThreads) {
        const uint4 gv = __ldcs(g + x);
        float4 a = t[2 * x], b = t[2 * x + 1];
        add8(a, b, gv);
        t[2 * x] = a; t[2 * x + 1] = b;
      }
    }
    __syncthreads();  // the lists are rewritten next round
    cur = nxt; cur_r = nxt_r;
  }
}

// ---- frequent ids ----------------------------------------------------------------------------------
// A table row that many rows add to (natural token streams have a Zipf-like head) would serialise on the one CTA
// that owns it.  Ids with at least `threshold` rows are taken out of k_embed_grad: their rows are listed in
// ascending order (a stable multi-way split of the row ids), and k_embed_grad_hot gives every (id, 256-column
// slice) its own CTA, which streams the listed rows through shared memory, eight warps loading, one warp adding in
// list order.  The order of additions per element is the same as on the other path: results do not depend on
// which path an id takes.
constexpr uint32_t kMaxHot = 512;       // at most this many ids take the hot path (the first by id if more qualify)
constexpr uint32_t kHotBlockRows = 256; // rows per CTA in the split kernels

struct HotArgs {
  uint64_t rows;
  uint32_t vocab, threshold, n_blocks;
  const int32_t* row_id;  // [rows]
  const uint32_t* id_count;  // [vocab]
  int32_t* hot_index;     // [vocab]: index among the hot ids, or -1
  int32_t* hot_ids;       // [kMaxHot]
  uint32_t* hot_off;      // [kMaxHot + 1]: first entry of each hot id's list
  uint32_t* n_hot;        // scalar
  uint32_t* blk_cnt;      // [kMaxHot + 1][n_blocks]: rows of hot id h (last: of no hot id) in row block b, then their exclusive scan
  uint32_t* hot_rows;     // [rows]: the lists, concatenated
  uint32_t* cold_row;     // [rows]: the other adding rows, ascending (what k_embed_grad walks)
  int32_t* cold_id;       // [rows]: their table rows
  uint32_t* n_cold;       // scalar
};

// one CTA: the first kMaxHot ids (in ascending id order) with at least `threshold` rows; they are then numbered by
// descending row count (ties by id), so the longest lists are started first; and where each list starts
__global__ void __launch_bounds__(1024) k_hot_select(HotArgs a) {
  __shared__ int32_t s_ids[kMaxHot];
  __shared__ uint32_t s_cnt[kMaxHot], s_sorted[kMaxHot];
  static_assert(kMaxHot <= 1024, "one thread per frequent id below");
  // thread t looks at the ids [t * per, (t + 1) * per): one scan over the threads' counts keeps id order
  const uint32_t per = (a.vocab + blockDim.x - 1) / blockDim.x;
  const uint32_t v0 = threadIdx.x * per, v1 = min(a.vocab, v0 + per);
  uint32_t mine = 0;
  for (uint32_t v = v0; v < v1; ++v) {
    const uint32_t c = a.id_count[v];
    mine += c >= a.threshold && c > 0;
    a.hot_index[v] = -1;
  }
  uint64_t tot;
  uint32_t idx = (uint32_t)block_exclusive_scan(mine, &tot);
  if (mine && idx < kMaxHot) {
    for (uint32_t v = v0; v < v1 && idx < kMaxHot; ++v) {
      const uint32_t c = a.id_count[v];
      if (c >= a.threshold && c > 0) { s_ids[idx] = (int32_t)v; s_cnt[idx] = c; ++idx; }
    }
  }
  __syncthreads();
  const uint32_t n = min((uint32_t)tot, kMaxHot);
  const uint32_t i = threadIdx.x;
  if (i < n) {
    uint32_t rank = 0;
    for (uint32_t j = 0; j < n; ++j) rank += (s_cnt[j] > s_cnt[i]) || (s_cnt[j] == s_cnt[i] && j < i);
    a.hot_ids[rank] = s_ids[i];
    a.hot_index[s_ids[i]] = (int32_t)rank;
    s_sorted[rank] = s_cnt[i];
  }
  __syncthreads();
  uint64_t total;
  const uint64_t ex = block_exclusive_scan(i < n ? s_sorted[i] : 0, &total);
  if (i < n) a.hot_off[i] = (uint32_t)ex;
  if (i == 0) { a.hot_off[n] = (uint32_t)total; *a.n_hot = n; }
}

// rows of each hot id, and adding rows of no hot id, per block of 256 rows
__global__ void __launch_bounds__(kHotBlockRows) k_split_count(HotArgs a) {
  const uint32_t n_hot = *a.n_hot;
  __shared__ uint32_t cnt[kMaxHot + 1];
  for (uint32_t h = threadIdx.x; h < n_hot; h += blockDim.x) cnt[h] = 0;
  if (threadIdx.x == 0) cnt[kMaxHot] = 0;
  __syncthreads();
  const uint64_t R = (uint64_t)blockIdx.x * kHotBlockRows + threadIdx.x;
  if (R < a.rows) {
    const int32_t id = a.row_id[R];
    if (id >= 0) {
      const int32_t h = a.hot_index[id];
      atomicAdd(&cnt[h >= 0 ? h : (int32_t)kMaxHot], 1u);
    }
  }
  __syncthreads();
  for (uint32_t h = threadIdx.x; h < n_hot; h += blockDim.x) a.blk_cnt[(uint64_t)h * a.n_blocks + blockIdx.x] = cnt[h];
  if (threadIdx.x == 0) a.blk_cnt[(uint64_t)kMaxHot * a.n_blocks + blockIdx.x] = cnt[kMaxHot];
}

// CTA h: exclusive scan of one list's per-block counts, offset by the start of the list (CTA kMaxHot: the cold list)
__global__ void __launch_bounds__(1024) k_split_scan(HotArgs a) {
  const uint32_t h = blockIdx.x;
  if (h != kMaxHot && h >= *a.n_hot) return;
  uint32_t* c = a.blk_cnt + (uint64_t)h * a.n_blocks;
  const uint32_t start = h == kMaxHot ? 0 : a.hot_off[h];
  uint64_t carry = 0;
  for (uint32_t b0 = 0; b0 < a.n_blocks; b0 += blockDim.x) {
    const uint32_t b = b0 + threadIdx.x;
    const uint64_t x = b < a.n_blocks ? c[b] : 0;
    uint64_t tot;
    const uint64_t ex = block_exclusive_scan(x, &tot);
    if (b < a.n_blocks) c[b] = start + (uint32_t)(carry + ex);
    carry += tot;
  }
  if (h == kMaxHot && threadIdx.x == 0) *a.n_cold = (uint32_t)carry;
}

// stable placement: a row goes behind the rows of the same list in earlier blocks, earlier warps, earlier lanes
__global__ void __launch_bounds__(kHotBlockRows) k_split_fill(HotArgs a) {
  const uint32_t n_hot = *a.n_hot;
  __shared__ uint32_t wc[kHotBlockRows / 32][kMaxHot];
  __shared__ uint32_t wcold[kHotBlockRows / 32];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (uint32_t i = threadIdx.x; i < (kHotBlockRows / 32) * n_hot; i += blockDim.x) wc[i / n_hot][i % n_hot] = 0;
  __syncthreads();
  const uint64_t R = (uint64_t)blockIdx.x * kHotBlockRows + threadIdx.x;
  int32_t id = -1, h = -1;
  if (R < a.rows) {
    id = a.row_id[R];
    if (id >= 0) h = a.hot_index[id];
  }
  const bool cold = id >= 0 && h < 0;
  const uint32_t lt = (1u << lane) - 1;
  const uint32_t cold_mask = __ballot_sync(0xFFFFFFFFu, cold);
  const uint32_t peers = __match_any_sync(0xFFFFFFFFu, h);
  const uint32_t rank = cold ? __popc(cold_mask & lt) : __popc(peers & lt);
  if (h >= 0 && rank == 0) wc[warp][h] = __popc(peers);
  if (lane == 0) wcold[warp] = __popc(cold_mask);
  __syncthreads();
  if (h >= 0) {
    uint32_t before = 0;
    for (uint32_t w = 0; w < warp; ++w) before += wc[w][h];
    a.hot_rows[a.blk_cnt[(uint64_t)h * a.n_blocks + blockIdx.x] + before + rank] = (uint32_t)R;
  } else if (cold) {
    uint32_t before = 0;
    for (uint32_t w = 0; w < warp; ++w) before += wcold[w];
    const uint32_t at = a.blk_cnt[(uint64_t)kMaxHot * a.n_blocks + blockIdx.x] + before + rank;
    a.cold_row[at] = (uint32_t)R;
    a.cold_id[at] = id;
  }
}

constexpr uint32_t kHotBatch = 32;   // rows per round: four per warp
constexpr uint32_t kHotStages = 6;   // staging buffers: rounds r+1 .. r+4 are in flight while round r is added
constexpr uint32_t kHotSmemBytes = kHotStages * kHotBatch * 32 * sizeof(uint4);  // 96 KiB

__device__ __forceinline__ void async_copy16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void async_wait_pending() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr uint32_t kHotThreads = 288;  // warp 0 adds; warps 1..8 fetch, four rows each per round

// CTA (s, h): columns [256 s, 256 s + 256) of hot id h.  The listed rows' slices flow through a ring of staging
// buffers filled by asynchronous 16-byte copies issued by the eight fetching warps (nobody waits on a register; the
// list entries of the next round are read a round ahead); warp 0 adds the staged rows in list order.  One barrier
// per round of 32 rows.
__global__ void __launch_bounds__(kHotThreads) k_embed_grad_hot(HotArgs a, uint32_t H, const uint4* __restrict__ grad, float* table) {
  extern __shared__ __align__(16) uint4 stage[];  // [kHotStages][kHotBatch][32]
  const uint32_t s = blockIdx.x, h = blockIdx.y;
  if (h >= *a.n_hot) return;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t vec_per_row = H >> 3, x = s * 32 + lane;
  const bool col = x < vec_per_row;
  const int32_t id = a.hot_ids[h];
  const uint32_t n = a.hot_off[h + 1] - a.hot_off[h];
  const uint32_t rounds = (n + kHotBatch - 1) / kHotBatch;
  const uint32_t* list = a.hot_rows + a.hot_off[h];
  if (warp == 0) {
    float4* t = reinterpret_cast<float4*>(table + (uint64_t)id * H);
    float4 acc_a = make_float4(0, 0, 0, 0), acc_b = acc_a;
    if (col) { acc_a = t[2 * x]; acc_b = t[2 * x + 1]; }
    for (uint32_t r = 0; r < rounds; ++r) {
      __syncthreads();  // round r is staged (the fetching warps waited for their copies before this barrier)
      if (col) {
        const uint4* buf = stage + (size_t)(r % kHotStages) * kHotBatch * 32;
        const uint32_t m = min(kHotBatch, n - r * kHotBatch);
        if (m == kHotBatch) {  // full round: the shared-memory reads of eight rows go out ahead of their additions
#pragma unroll 8
          for (uint32_t i = 0; i < kHotBatch; ++i) add8(acc_a, acc_b, buf[i * 32 + lane]);
        } else {
          for (uint32_t i = 0; i < m; ++i) add8(acc_a, acc_b, buf[i * 32 + lane]);
        }
      }
    }
    if (col) { t[2 * x] = acc_a; t[2 * x + 1] = acc_b; }
    return;
  }
  const uint32_t j0 = (warp - 1) * (kHotBatch / 8);  // this warp's rows inside a round
  uint32_t idx[kHotBatch / 8];
  auto read_list = [&](uint32_t r) {
#pragma unroll
    for (uint32_t i = 0; i < kHotBatch / 8; ++i) {
      const uint32_t k = r * kHotBatch + j0 + i;
      idx[i] = k < n ? list[k] : 0;
    }
  };
  auto issue_round = [&](uint32_t r) {  // this thread's copies of round r, as one group (empty past the end)
    if (r < rounds && col) {
      uint4* buf = stage + (size_t)(r % kHotStages) * kHotBatch * 32;
#pragma unroll
      for (uint32_t i = 0; i < kHotBatch / 8; ++i)
        if (r * kHotBatch + j0 + i < n) async_copy16(buf + (j0 + i) * 32 + lane, grad + (uint64_t)idx[i] * vec_per_row + x);
    }
    async_commit();
  };
  for (uint32_t r = 0; r + 2 < kHotStages; ++r) { read_list(r); issue_round(r); }  // rounds 0 .. kHotStages-3
  read_list(kHotStages - 2);
  for (uint32_t r = 0; r < rounds; ++r) {
    async_wait_pending<kHotStages - 3>();  // this thread's copies of round r have landed
    __syncthreads();                       // everyone's have; and warp 0 is done with round r-1
    issue_round(r + kHotStages - 2);       // into the buffer of round r-2, free since the barrier before this one
    read_list(r + kHotStages - 1);         // needed one round from now
  }
  async_wait_pending<0>();
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
  // a span named more than once keeps its last grid: only that item is uploaded (the kernel writes in parallel)
  std::vector<uint32_t> keep;
  {
    std::unordered_set<uint32_t> seen;
    for (uint32_t i = n; i-- > 0;)
      if (seen.insert(slot[i] * S + span_idx[i]).second) keep.push_back(i);
  }
  n = (uint32_t)keep.size();
  const size_t o_grid = 0, o_sid = align_up_sz((size_t)n * sizeof(uint4), 16), bytes = o_sid + (size_t)n * 4;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ft_call_ctx* cx = nullptr;
  int32_t rc = ctx_acquire(p, 0, bytes, bytes, &cx);
  if (rc != FT_OK) return rc;
  uint4* hg = reinterpret_cast<uint4*>(static_cast<uint8_t*>(cx->h) + o_grid);
  uint32_t* hs = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(cx->h) + o_sid);
  for (uint32_t k = 0; k < n; ++k) {
    const uint32_t i = keep[k];
    hg[k] = make_uint4(grid_thw[3ull * i], grid_thw[3ull * i + 1], grid_thw[3ull * i + 2], 0);
    hs[k] = slot[i] * S + span_idx[i];
  }
  for (uint32_t k = 0; k < n; ++k) memcpy(p->spans[hs[k]].grid, &hg[k], 12);  // host mirror (exported with the sample)
  if ((rc = ctx_upload(p, cx, bytes)) != FT_OK) return rc;
  // assemblies already in flight on a caller's stream read the grids as they were: the metadata stream waits for them
  if ((rc = meta_after_data(p)) != FT_OK) return rc;
  if ((rc = meta_after(p, st)) != FT_OK) return rc;
  GridCall c;
  c.n = n;
  c.grid = reinterpret_cast<const uint4*>(static_cast<uint8_t*>(cx->d) + o_grid);
  c.span_id = reinterpret_cast<const uint32_t*>(static_cast<uint8_t*>(cx->d) + o_sid);
  k_set_grids<<<(n + 255) / 256, 256, 0, p->meta>>>(p->view, c);
  FT_CUDA(cudaGetLastError());
  if ((rc = ctx_release(p, cx, p->meta)) != FT_OK) return rc;
  p->gpu_launches += 1;
  if ((rc = meta_to(p, st)) != FT_OK) return rc;
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
    ft_call_ctx* cx = nullptr;
    int32_t rc1 = ctx_acquire(p, 1, 0, 0, &cx, false, st);  // for its claim counter
    if (rc1 != FT_OK) return rc1;
    rc1 = gather_launch(p, pl, mb_begin, mb_end, embed_table, vocab, out_embeds, nullptr, nullptr, lay.L, st, nullptr, 0, 0, 0, cx->counters);
    if (rc1 != FT_OK) return rc1;
    if ((rc1 = ctx_release(p, cx, st)) != FT_OK) return rc1;
  }
  const PlanView pv = make_plan_view(pl);
  k_pad_zero<<<(unsigned)p->sm_count * 8, 256, 0, st>>>(pv, lay, p->view.row_bytes, static_cast<uint8_t*>(out_embeds));
  IndexArgs ia;
  ia.lay = lay; ia.pad_id = pad_id; ia.cu = out_cu; ia.pos3 = out_pos3; ia.ids = out_ids; ia.labels = out_labels;
  ia.mask = out_mask; ia.call_seq = status_seq(p);
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
  if (!p->grad_attr_set) {  // once per pool, hence once per device the pool lives on
    FT_CUDA(cudaFuncSetAttribute(k_embed_grad_hot, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHotSmemBytes));
    p->grad_attr_set = true;
  }
  // one stream-ordered scratch block: row ids, per-id counts, and the tables of the frequent-id path
  const uint32_t ctas = std::min<uint32_t>(vocab, (uint32_t)p->sm_count * (uint32_t)p->grad_ctas_per_sm);
  const uint32_t n_blocks = (uint32_t)((lay.rows + kHotBlockRows - 1) / kHotBlockRows);
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t o = off; off = align_up_sz(off + bytes, 256); return o; };
  const size_t o_row = take((lay.rows + 4) * 4), o_cnt = take((size_t)vocab * 4), o_hidx = take((size_t)vocab * 4);
  const size_t o_hids = take(kMaxHot * 4), o_hoff = take((kMaxHot + 1) * 4), o_nhot = take(4);
  const size_t o_blk = take((size_t)(kMaxHot + 1) * n_blocks * 4), o_hrows = take(lay.rows * 4);
  const size_t o_crow = take((lay.rows + 4) * 4), o_cid = take((lay.rows + 4) * 4), o_ncold = take(4);
  uint8_t* d = nullptr;
  FT_CUDA(cudaMallocAsync(reinterpret_cast<void**>(&d), off, st));
  RowIdArgs ra;
  ra.lay = lay; ra.vocab = vocab; ra.row_id = reinterpret_cast<int32_t*>(d + o_row);
  ra.id_count = reinterpret_cast<uint32_t*>(d + o_cnt); ra.call_seq = status_seq(p);
  HotArgs ha;
  ha.rows = lay.rows; ha.vocab = vocab; ha.n_blocks = n_blocks;
  // an id is frequent when its rows alone are an eighth of an average CTA's share of the layout's rows
  ha.threshold = p->grad_hot_threshold ? (uint32_t)p->grad_hot_threshold : (uint32_t)std::max<uint64_t>(64, lay.rows / (8ull * ctas));
  ha.row_id = ra.row_id; ha.id_count = ra.id_count;
  ha.hot_index = reinterpret_cast<int32_t*>(d + o_hidx); ha.hot_ids = reinterpret_cast<int32_t*>(d + o_hids);
  ha.hot_off = reinterpret_cast<uint32_t*>(d + o_hoff); ha.n_hot = reinterpret_cast<uint32_t*>(d + o_nhot);
  ha.blk_cnt = reinterpret_cast<uint32_t*>(d + o_blk); ha.hot_rows = reinterpret_cast<uint32_t*>(d + o_hrows);
  ha.cold_row = reinterpret_cast<uint32_t*>(d + o_crow); ha.cold_id = reinterpret_cast<int32_t*>(d + o_cid);
  ha.n_cold = reinterpret_cast<uint32_t*>(d + o_ncold);
  const PlanView pv = make_plan_view(pl);
  const uint32_t H = p->view.hidden, slices = ((H >> 3) + 31) / 32;
  cudaError_t e = cudaMemsetAsync(ra.id_count, 0, (size_t)vocab * 4, st);
  if (e == cudaSuccess) {
    prof_begin(p, FT_K_EMBED_GRAD, st);
    k_grad_row_ids<<<(unsigned)((lay.rows + 255) / 256), 256, 0, st>>>(p->view, pv, ra);
    k_hot_select<<<1, 1024, 0, st>>>(ha);
    k_split_count<<<n_blocks, kHotBlockRows, 0, st>>>(ha);
    k_split_scan<<<kMaxHot + 1, 1024, 0, st>>>(ha);
    k_split_fill<<<n_blocks, kHotBlockRows, 0, st>>>(ha);
    // the two adding kernels touch disjoint table rows: the frequent-id one runs beside the other on the
    // consumer side's second stream
    cudaEventRecord(p->fork_ev[1], st);
    cudaStreamWaitEvent(p->side_stream[1], p->fork_ev[1], 0);
    k_embed_grad<<<ctas, kGradThreads, 0, st>>>(ha.cold_id, ha.cold_row, ha.n_cold, H, static_cast<const uint4*>(grad_out), grad_table);
    k_embed_grad_hot<<<dim3(slices, kMaxHot), kHotThreads, kHotSmemBytes, p->side_stream[1]>>>(ha, H, static_cast<const uint4*>(grad_out), grad_table);
    cudaEventRecord(p->join_ev[1], p->side_stream[1]);
    cudaStreamWaitEvent(st, p->join_ev[1], 0);
    prof_end(p, st);
    e = cudaGetLastError();
  }
  cudaFreeAsync(d, st);
  if (e != cudaSuccess) return cuda_fail(e, "pool_embed_grad");
  p->gpu_launches += 7;
  const_cast<ft_plan*>(pl)->last_stream = st;
  return end_consumer(p, st);
}
