// The dynamic packing rule on the device (Sec. 3.4, Algorithm 1, Eq. 3).
//
// Kernels in this file
//   k_plan_prepare   l(s) from the pool's sample table, per-sample score (Eq. 3 on a singleton)
//   k_bestfit        Algorithm 1 lines 1-11: online best fit.  The paper's segment tree over [0, L]
//                    becomes a 32-ary bitmap hierarchy in shared memory (find-next-set = best-fit query,
//                    same answer, O(log_32 L)); per-residual LIFO stacks give the tie rule.
//   k_pack_order     packing order: the caller's, or longest first (variant), by counting
//   k_mb_finalize    exclusive scans -> mb_sample_off, mb_row_off
//   k_plan_scatter   samples into microbatch-major, append order
//   k_mb_cost        Cost(B_j) (lmax^2 as printed, or the sum-of-squares variant), min/max cost
//   k_row_offsets    exclusive scan of lengths in plan order
//   k_tiles          plan position of the sample holding each 32-row output tile
//   k_bucket         lines 12-14: equal-width cost buckets
//   k_sort_deal      lines 15-27: rank-by-counting sort (bucket desc, cost desc, index asc), zig-zag deal
//   k_rank_index/_scan/_lists  per-rank lists in dispatch order
#include <algorithm>
#include <cstring>

#include "flowpool_internal.cuh"

namespace ft {

struct MbRec { uint32_t residual, lmax, count, next; };

constexpr uint32_t kFitChunk = 2048;  // samples staged through shared memory per round
enum { SC_NMB = 0, SC_MAXTOK = 1, SC_TOTAL_LO = 2, SC_TOTAL_HI = 3, SC_LO = 4, SC_HI = 6, SC_COUNT = 8 };

__global__ void k_plan_prepare(PoolView v, const uint32_t* slots, uint32_t n, uint64_t A, uint64_t B, uint32_t* len,
                               uint64_t* sample_cost) {
  const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const uint64_t l = v.s_seq_len[slots[t]];  // l(s): the LLM-side length, text + all vision tokens
  len[t] = (uint32_t)l;
  sample_cost[t] = A * l + B * l * l;
}

// Packing order.  Default: the caller's order.  Variant (longest first): position of sample t = number of
// samples that are longer, or equally long and earlier -- rank by counting, tiles of lengths through shared memory.
__global__ void __launch_bounds__(256) k_pack_order(const uint32_t* __restrict__ len, uint32_t n, uint32_t sort_desc,
                                                    uint32_t* pk_t, uint32_t* pk_len) {
  __shared__ uint32_t tile[1024];
  const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t lt = t < n ? len[t] : 0;
  uint32_t r = t;
  if (sort_desc) {
    r = 0;
    for (uint32_t base = 0; base < n; base += 1024) {
      const uint32_t cnt = min(1024u, n - base);
      __syncthreads();
      for (uint32_t i = threadIdx.x; i < cnt; i += blockDim.x) tile[i] = len[base + i];
      __syncthreads();
      if (t < n)
        for (uint32_t i = 0; i < cnt; ++i) r += (tile[i] > lt) || (tile[i] == lt && base + i < t);
    }
  }
  if (t < n) { pk_t[r] = t; pk_len[r] = lt; }
}

// Residual bitmap: bit r of level 0 is set when some open microbatch has residual r; bit i of level k+1 is set
// when word i of level k is non-zero.  Four levels of 32-ary words cover residuals below 2^20.  The levels live in
// the kernel's shared memory and are addressed by word offsets from its base; every level carries one zero word
// of padding behind its last word, so the query needs no bounds checks.
struct FitOff {
  uint32_t b0, b1, b2, b3;  // word offsets of the levels
};

// smallest set index >= l, or kNone: the best-fit query (the segment-tree descent of Algorithm 1, 32-ary)
__device__ __forceinline__ uint32_t fit_find(const uint32_t* sm, const FitOff f, uint32_t l) {
  uint32_t w = l >> 5;
  uint32_t m = sm[f.b0 + w] & (0xFFFFFFFFu << (l & 31));
  if (m) return (w << 5) + __ffs(m) - 1;
  const uint32_t i1 = w + 1;
  w = i1 >> 5;
  m = sm[f.b1 + w] & (0xFFFFFFFFu << (i1 & 31));
  if (m) {
    const uint32_t p0 = (w << 5) + __ffs(m) - 1;
    return (p0 << 5) + __ffs(sm[f.b0 + p0]) - 1;
  }
  const uint32_t i2 = w + 1;
  w = i2 >> 5;
  m = sm[f.b2 + w] & (0xFFFFFFFFu << (i2 & 31));
  if (m) {
    const uint32_t p1 = (w << 5) + __ffs(m) - 1;
    const uint32_t p0 = (p1 << 5) + __ffs(sm[f.b1 + p1]) - 1;
    return (p0 << 5) + __ffs(sm[f.b0 + p0]) - 1;
  }
  const uint32_t i3 = w + 1;
  w = i3 >> 5;
  m = sm[f.b3 + w] & (0xFFFFFFFFu << (i3 & 31));
  if (m) {
    const uint32_t p2 = (w << 5) + __ffs(m) - 1;
    const uint32_t p1 = (p2 << 5) + __ffs(sm[f.b2 + p2]) - 1;
    const uint32_t p0 = (p1 << 5) + __ffs(sm[f.b1 + p1]) - 1;
    return (p0 << 5) + __ffs(sm[f.b0 + p0]) - 1;
  }
  return kNone;
}
__device__ __forceinline__ void fit_set(uint32_t* sm, const FitOff f, uint32_t r) {
  uint32_t old = sm[f.b0 + (r >> 5)];
  sm[f.b0 + (r >> 5)] = old | (1u << (r & 31));
  if (old) return;
  r >>= 5; old = sm[f.b1 + (r >> 5)]; sm[f.b1 + (r >> 5)] = old | (1u << (r & 31));
  if (old) return;
  r >>= 5; old = sm[f.b2 + (r >> 5)]; sm[f.b2 + (r >> 5)] = old | (1u << (r & 31));
  if (old) return;
  r >>= 5; sm[f.b3 + (r >> 5)] |= 1u << (r & 31);
}
__device__ __forceinline__ void fit_clear(uint32_t* sm, const FitOff f, uint32_t r) {
  uint32_t nw = sm[f.b0 + (r >> 5)] & ~(1u << (r & 31));
  sm[f.b0 + (r >> 5)] = nw;
  if (nw) return;
  r >>= 5; nw = sm[f.b1 + (r >> 5)] & ~(1u << (r & 31)); sm[f.b1 + (r >> 5)] = nw;
  if (nw) return;
  r >>= 5; nw = sm[f.b2 + (r >> 5)] & ~(1u << (r & 31)); sm[f.b2 + (r >> 5)] = nw;
  if (nw) return;
  r >>= 5; sm[f.b3 + (r >> 5)] &= ~(1u << (r & 31));
}

// One block.  Thread 0 walks the samples in order (the dependency chain of online best fit); the other
// threads stage lengths in and results out, coalesced, and initialise / flush the tables.
// HEAD_SMEM: the per-residual stack heads live in shared memory (budgets up to about 32 K), else in global.
// RECS_SMEM: every microbatch record fits in shared memory (else those past rec_smem_cap live in global).
template <bool HEAD_SMEM, bool RECS_SMEM>
__global__ void __launch_bounds__(1024) k_bestfit(const uint32_t* __restrict__ len, uint32_t n, uint32_t L,
                                                  uint32_t* __restrict__ head_g, MbRec* __restrict__ recs_g,
                                                  uint32_t rec_smem_cap, uint32_t* sample_mb, uint32_t* sample_rank,
                                                  uint32_t* mb_residual, uint32_t* mb_tokens, uint32_t* mb_lmax,
                                                  uint32_t* mb_count, uint32_t* scalars) {
  extern __shared__ __align__(16) uint32_t sm[];
  FitOff f;
  uint32_t o = 0;
  const uint32_t w0 = (L + 1 + 31) / 32, w1 = (w0 + 31) / 32, w2 = (w1 + 31) / 32, w3 = (w2 + 31) / 32;
  f.b0 = o; o += w0 + 1;
  f.b1 = o; o += w1 + 1;
  f.b2 = o; o += w2 + 1;
  f.b3 = o; o += w3 + 1;
  const uint32_t total_words = o;
  const uint32_t o_len = o; o += kFitChunk;
  const uint32_t o_mb = o; o += kFitChunk;
  const uint32_t o_rank = o; o += kFitChunk;
  const uint32_t o_head = o;
  if (HEAD_SMEM) o += L + 1;
  o = (o + 3) & ~3u;  // 16-byte align the records
  uint4* recs_s = reinterpret_cast<uint4*>(sm + o);
  uint4* recs_gv = reinterpret_cast<uint4*>(recs_g);

  for (uint32_t i = threadIdx.x; i < total_words; i += blockDim.x) sm[i] = 0;
  if (HEAD_SMEM) { for (uint32_t i = threadIdx.x; i <= L; i += blockDim.x) sm[o_head + i] = kNone; }
  else { for (uint32_t i = threadIdx.x; i <= L; i += blockDim.x) head_g[i] = kNone; }
  __shared__ uint32_t s_nmb;
  if (threadIdx.x == 0) s_nmb = 0;
  __syncthreads();

  auto head_ld = [&](uint32_t r) -> uint32_t { return HEAD_SMEM ? sm[o_head + r] : head_g[r]; };
  auto head_st = [&](uint32_t r, uint32_t v) { if (HEAD_SMEM) sm[o_head + r] = v; else head_g[r] = v; };
  // a record: x = residual, y = lmax, z = count, w = next (the MbRec layout)
  auto rec_ld = [&](uint32_t j) -> uint4 { return (RECS_SMEM || j < rec_smem_cap) ? recs_s[j] : recs_gv[j]; };
  auto rec_st = [&](uint32_t j, uint4 v) { if (RECS_SMEM || j < rec_smem_cap) recs_s[j] = v; else recs_gv[j] = v; };

  for (uint32_t base = 0; base < n; base += kFitChunk) {
    const uint32_t cnt = min(kFitChunk, n - base);
    for (uint32_t i = threadIdx.x; i < cnt; i += blockDim.x) sm[o_len + i] = len[base + i];
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t n_mb = s_nmb;
      for (uint32_t i = 0; i < cnt; ++i) {
        const uint32_t l = sm[o_len + i];
        const uint32_t r = fit_find(sm, f, l);  // the smallest residual >= l among open microbatches
        uint32_t j;
        uint4 rec;
        if (r != kNone) {
          j = head_ld(r);  // most recently changed microbatch with that residual
          rec = rec_ld(j);
          head_st(r, rec.w);
          if (rec.w == kNone) fit_clear(sm, f, r);
          rec.x = r - l;
          rec.y = max(rec.y, l);
          rec.z++;
        } else {
          j = n_mb++;
          rec.x = L - l; rec.y = l; rec.z = 1;
        }
        // a residual of 0 can never be chosen again (l >= 1): it needs no stack entry
        if (rec.x) {
          rec.w = head_ld(rec.x);
          head_st(rec.x, j);
          if (rec.w == kNone) fit_set(sm, f, rec.x);
        } else {
          rec.w = kNone;
        }
        rec_st(j, rec);
        sm[o_mb + i] = j;
        sm[o_rank + i] = rec.z - 1;
      }
      s_nmb = n_mb;
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < cnt; i += blockDim.x) { sample_mb[base + i] = sm[o_mb + i]; sample_rank[base + i] = sm[o_rank + i]; }
    __syncthreads();
  }
  const uint32_t n_mb = s_nmb;
  for (uint32_t j = threadIdx.x; j < n_mb; j += blockDim.x) {
    const uint4 rec = rec_ld(j);
    mb_residual[j] = rec.x; mb_tokens[j] = L - rec.x; mb_lmax[j] = rec.y; mb_count[j] = rec.z;
  }
  if (threadIdx.x == 0) scalars[SC_NMB] = n_mb;
}

// Online best fit with a whole warp, for plans with few microbatches.  Every open microbatch has a 64-bit key,
// residual << 32 | ~stamp (stamp = the sample that changed it last): the smallest key among those whose residual is
// >= l is the smallest such residual and, among equal residuals, the most recently changed microbatch: the
// tie-break of the packing rule.  Stamps are distinct, so keys are.  Every lane looks at a 32nd of the keys and two
// warp reductions (high word, then low word among the lanes that hold the winning high word) find the winner.
// A step of the chain costs a few hundred cycles instead of the thousand of the bitmap descent with its per-residual
// stacks, and the kernels need little or no shared memory, so they also start on an SM whose shared-memory split was
// chosen for the copy kernels.  The caller bounds the microbatch count: any-fit packing leaves at most one microbatch
// half empty, so n_mb <= 2 sum(l) / L + 1.
constexpr uint32_t kWarpFitChunk = 256;
constexpr uint32_t kWarpFitMaxCap = 1024;
constexpr unsigned long long kNoKey = ~0ull;
__device__ __forceinline__ unsigned long long fit_key(uint32_t residual, uint32_t stamp) {
  return ((unsigned long long)residual << 32) | (0xFFFFFFFFu - stamp);
}
// the smallest key of the warp (kNoKey if no lane has one)
__device__ __forceinline__ unsigned long long warp_min_key(unsigned long long k) {
  const uint32_t hi = (uint32_t)(k >> 32), lo = (uint32_t)k;
  const uint32_t mh = __reduce_min_sync(0xFFFFFFFFu, hi);
  const uint32_t ml = __reduce_min_sync(0xFFFFFFFFu, hi == mh ? lo : 0xFFFFFFFFu);
  return ((unsigned long long)mh << 32) | ml;
}

// Keys in shared memory (8 bytes per microbatch, + 8 for lmax and count): up to kWarpFitMaxCap microbatches.
__global__ void __launch_bounds__(256) k_bestfit_warp(const uint32_t* __restrict__ len, uint32_t n, uint32_t L, uint32_t cap,
                                                      uint32_t* sample_mb, uint32_t* sample_rank, uint32_t* mb_residual,
                                                      uint32_t* mb_tokens, uint32_t* mb_lmax, uint32_t* mb_count, uint32_t* scalars) {
  extern __shared__ __align__(16) unsigned long long smk[];
  unsigned long long* key = smk;                                 // [cap]; kNoKey = not open
  uint32_t* lmax = reinterpret_cast<uint32_t*>(key + cap);       // [cap]
  uint32_t* cnt = lmax + cap;                                    // [cap]
  uint32_t *s_len = cnt + cap, *s_mb = s_len + kWarpFitChunk, *s_rank = s_mb + kWarpFitChunk;
  __shared__ uint32_t s_nmb;
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) s_nmb = 0;
  for (uint32_t base = 0; base < n; base += kWarpFitChunk) {
    const uint32_t c = min(kWarpFitChunk, n - base);
    for (uint32_t i = threadIdx.x; i < c; i += blockDim.x) s_len[i] = len[base + i];
    __syncthreads();
    if (warp == 0) {
      uint32_t n_mb = s_nmb;
      for (uint32_t i = 0; i < c; ++i) {
        const uint32_t l = s_len[i];
        const unsigned long long floor_key = (unsigned long long)l << 32;  // keys below it have a residual < l
        unsigned long long best = kNoKey;
        uint32_t bj = 0;
        for (uint32_t j0 = 0; j0 < n_mb; j0 += 128) {  // four independent loads per lane and round
          unsigned long long k[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t j = j0 + 32 * u + lane;
            k[u] = j < n_mb ? key[j] : kNoKey;
          }
#pragma unroll
          for (int u = 0; u < 4; ++u)
            if (k[u] >= floor_key && k[u] < best) { best = k[u]; bj = j0 + 32 * u + lane; }
        }
        const unsigned long long win = warp_min_key(best);
        if (win != kNoKey) {
          if (best == win) {  // keys are distinct: one lane
            key[bj] = fit_key((uint32_t)(win >> 32) - l, base + i);
            lmax[bj] = max(lmax[bj], l);
            const uint32_t k0 = cnt[bj];
            cnt[bj] = k0 + 1;
            s_mb[i] = bj; s_rank[i] = k0;
          }
        } else {
          if (lane == 0) {
            if (n_mb < cap) { key[n_mb] = fit_key(L - l, base + i); lmax[n_mb] = l; cnt[n_mb] = 1; }
            s_mb[i] = n_mb; s_rank[i] = 0;
          }
          if (n_mb < cap) ++n_mb;  // (the bound guarantees it)
        }
        __syncwarp();
      }
      if (lane == 0) s_nmb = n_mb;
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c; i += blockDim.x) { sample_mb[base + i] = s_mb[i]; sample_rank[base + i] = s_rank[i]; }
    __syncthreads();
  }
  const uint32_t n_mb = s_nmb;
  for (uint32_t j = threadIdx.x; j < n_mb; j += blockDim.x) {
    const uint32_t r = (uint32_t)(key[j] >> 32);
    mb_residual[j] = r; mb_tokens[j] = L - r; mb_lmax[j] = lmax[j]; mb_count[j] = cnt[j];
  }
  if (threadIdx.x == 0) scalars[SC_NMB] = n_mb;
}

// The same with the keys in registers, for plans of at most 32 R microbatches (microbatch j lives in slot j / 32 of
// lane j % 32): no memory access on the chain at all.
template <int R>
__global__ void __launch_bounds__(256) k_bestfit_regs(const uint32_t* __restrict__ len, uint32_t n, uint32_t L,
                                                      uint32_t* sample_mb, uint32_t* sample_rank, uint32_t* mb_residual,
                                                      uint32_t* mb_tokens, uint32_t* mb_lmax, uint32_t* mb_count, uint32_t* scalars) {
  __shared__ uint32_t s_len[kWarpFitChunk + 1], s_mb[kWarpFitChunk], s_rank[kWarpFitChunk];
  const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long K[R];  // kNoKey = not open (a full microbatch has residual 0 and is never >= l)
  uint32_t Lm[R], Cn[R];
#pragma unroll
  for (int s = 0; s < R; ++s) { K[s] = kNoKey; Lm[s] = 0; Cn[s] = 0; }
  uint32_t n_mb = 0;
  for (uint32_t base = 0; base < n; base += kWarpFitChunk) {
    const uint32_t c = min(kWarpFitChunk, n - base);
    for (uint32_t i = threadIdx.x; i < c; i += blockDim.x) s_len[i] = len[base + i];
    if (threadIdx.x == 0) s_len[c] = 0;
    __syncthreads();
    if (warp == 0) {
      uint32_t l_next = s_len[0];
      for (uint32_t i = 0; i < c; ++i) {
        const uint32_t l = l_next;
        l_next = s_len[i + 1];  // off the chain
        const unsigned long long floor_key = (unsigned long long)l << 32;
        unsigned long long cand[R];
#pragma unroll
        for (int s = 0; s < R; ++s) cand[s] = (K[s] >= floor_key && K[s] != kNoKey) ? K[s] : kNoKey;
#pragma unroll
        for (int w = 1; w < R; w <<= 1)  // pairwise minimum
#pragma unroll
          for (int s = 0; s + w < R; s += 2 * w) cand[s] = min(cand[s], cand[s + w]);
        const unsigned long long best = cand[0];
        const unsigned long long win = warp_min_key(best);
        if (win != kNoKey) {
          if (best == win) {  // keys are distinct: one lane, one slot
            const unsigned long long upd = fit_key((uint32_t)(win >> 32) - l, base + i);
            uint32_t k0 = 0, slot = 0;
#pragma unroll
            for (int s = 0; s < R; ++s)
              if (K[s] == win) { K[s] = upd; Lm[s] = max(Lm[s], l); k0 = Cn[s]; Cn[s] = k0 + 1; slot = s; }
            s_mb[i] = lane + 32u * slot;
            s_rank[i] = k0;
          }
        } else {
          if (lane == (n_mb & 31u)) {
            const int slot = (int)(n_mb >> 5);
#pragma unroll
            for (int s = 0; s < R; ++s)
              if (s == slot) { K[s] = fit_key(L - l, base + i); Lm[s] = l; Cn[s] = 1; }
            s_mb[i] = n_mb; s_rank[i] = 0;
          }
          ++n_mb;
        }
      }
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < c; i += blockDim.x) { sample_mb[base + i] = s_mb[i]; sample_rank[base + i] = s_rank[i]; }
    __syncthreads();
  }
  if (warp == 0) {
#pragma unroll
    for (int s = 0; s < R; ++s) {
      const uint32_t j = lane + 32u * (uint32_t)s;
      if (j < n_mb) {
        const uint32_t r = (uint32_t)(K[s] >> 32);
        mb_residual[j] = r; mb_tokens[j] = L - r; mb_lmax[j] = Lm[s]; mb_count[j] = Cn[s];
      }
    }
    if (lane == 0) scalars[SC_NMB] = n_mb;
  }
}

__global__ void __launch_bounds__(1024) k_mb_finalize(const uint32_t* mb_tokens, const uint32_t* mb_count,
                                                      uint32_t* mb_sample_off, uint64_t* mb_row_off, uint32_t* scalars) {
  __shared__ uint32_t s_max;
  const uint32_t n_mb = scalars[SC_NMB];
  if (threadIdx.x == 0) s_max = 0;
  __syncthreads();
  uint64_t cs = 0, cr = 0;
  for (uint32_t base = 0; base < n_mb; base += blockDim.x) {
    const uint32_t j = base + threadIdx.x;
    uint64_t cnt = 0, tok = 0;
    if (j < n_mb) {
      cnt = mb_count[j]; tok = mb_tokens[j];
      atomicMax(&s_max, (uint32_t)tok);
    }
    uint64_t ts, tr;
    const uint64_t es = block_exclusive_scan(cnt, &ts);
    const uint64_t er = block_exclusive_scan(tok, &tr);
    if (j < n_mb) { mb_sample_off[j] = (uint32_t)(cs + es); mb_row_off[j] = cr + er; }
    cs += ts; cr += tr;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    mb_sample_off[n_mb] = (uint32_t)cs; mb_row_off[n_mb] = cr;
    scalars[SC_MAXTOK] = s_max;
    scalars[SC_TOTAL_LO] = (uint32_t)cr; scalars[SC_TOTAL_HI] = (uint32_t)(cr >> 32);
    *reinterpret_cast<unsigned long long*>(scalars + SC_LO) = ~0ull;  // cost range, filled by k_mb_cost
    *reinterpret_cast<unsigned long long*>(scalars + SC_HI) = 0;
  }
}

// Cost(B_j), lines 12-14: A * sum(l) + B * lmax^2 (Eq. 3 times L^2 when (A, B) = (L, 1)); variant: B * sum(l^2).
__global__ void k_mb_cost(uint64_t A, uint64_t B, uint32_t sumsq, const uint32_t* mb_tokens, const uint32_t* mb_lmax,
                          const uint32_t* mb_sample_off, const uint64_t* plan_len, uint64_t* mb_cost, uint32_t* scalars) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= scalars[SC_NMB]) return;
  uint64_t quad;
  if (sumsq) {
    quad = 0;
    for (uint32_t q = mb_sample_off[j]; q < mb_sample_off[j + 1]; ++q) quad += plan_len[q] * plan_len[q];
  } else {
    const uint64_t lm = mb_lmax[j];
    quad = lm * lm;
  }
  const uint64_t cost = A * mb_tokens[j] + B * quad;
  mb_cost[j] = cost;
  atomicMin(reinterpret_cast<unsigned long long*>(scalars + SC_LO), (unsigned long long)cost);
  atomicMax(reinterpret_cast<unsigned long long*>(scalars + SC_HI), (unsigned long long)cost);
}

__global__ void k_plan_scatter(const uint32_t* slots, const uint32_t* pk_t, const uint32_t* pk_len, const uint32_t* pk_mb,
                               const uint32_t* pk_rank, const uint32_t* mb_sample_off, uint32_t n, uint32_t* mb_samples,
                               uint64_t* plan_len, uint32_t* plan_sample_mb, uint32_t* sample_mb) {
  const uint32_t r = blockIdx.x * blockDim.x + threadIdx.x;  // packing position
  if (r >= n) return;
  const uint32_t j = pk_mb[r], q = mb_sample_off[j] + pk_rank[r];  // append order = packing order
  const uint32_t t = pk_t[r];
  mb_samples[q] = slots[t];
  plan_len[q] = pk_len[r];
  plan_sample_mb[q] = j;
  sample_mb[t] = j;
}

__global__ void __launch_bounds__(1024) k_row_offsets(const uint64_t* plan_len, uint32_t n, uint64_t* sample_row_off) {
  uint64_t carry = 0;
  for (uint32_t base = 0; base < n; base += blockDim.x) {
    const uint32_t q = base + threadIdx.x;
    uint64_t total;
    const uint64_t ex = block_exclusive_scan(q < n ? plan_len[q] : 0, &total);
    if (q < n) sample_row_off[q] = carry + ex;
    carry += total;
  }
  if (threadIdx.x == 0) sample_row_off[n] = carry;
}

// one thread per 32-row tile: the plan position of the sample holding the tile's first row (last q with
// sample_row_off[q] <= 32 t; samples are never empty)
__global__ void k_tiles(const uint64_t* sample_row_off, uint32_t n, uint64_t n_tiles, uint32_t* tile_first_sample) {
  const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n_tiles) return;
  const uint64_t row = t * 32;
  if (row >= sample_row_off[n]) return;  // the spare entry past the last row
  uint32_t lo = 0, hi = n;
  while (hi - lo > 1) {
    const uint32_t mid = (lo + hi) >> 1;
    if (sample_row_off[mid] <= row) lo = mid; else hi = mid;
  }
  tile_first_sample[t] = lo;
}

// auto_N != 0 (variant): K is only the upper limit; one bucket per full zig-zag round trip of 2N microbatches.
__global__ void k_bucket(const uint64_t* mb_cost, uint32_t K, uint32_t auto_N, const uint32_t* scalars, uint32_t* mb_bucket) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t n_mb = scalars[SC_NMB];
  if (j >= n_mb) return;
  if (auto_N) {
    const unsigned long long trips = max(1ull, ((unsigned long long)n_mb + 2ull * auto_N - 1) / (2ull * auto_N));
    if (trips < K) K = (uint32_t)trips;
  }
  const uint64_t lo = *reinterpret_cast<const unsigned long long*>(scalars + SC_LO);
  const uint64_t hi = *reinterpret_cast<const unsigned long long*>(scalars + SC_HI);
  const unsigned __int128 num = (unsigned __int128)(mb_cost[j] - lo) * K;
  mb_bucket[j] = (uint32_t)(num / ((unsigned __int128)(hi - lo) + 1));
}

// Sorted position by counting: i comes before j when its bucket is higher, or equal bucket and cost higher,
// or both equal and i < j.  Position inside the bucket -> zig-zag rank: round a/N forward when even.
__global__ void k_sort_deal(const uint64_t* mb_cost, const uint32_t* mb_bucket, uint32_t N, uint32_t carry,
                            const uint32_t* scalars, uint32_t* mb_pos, uint32_t* mb_rank) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t n_mb = scalars[SC_NMB];
  if (j >= n_mb) return;
  const uint64_t cj = mb_cost[j];
  const uint32_t bj = mb_bucket[j];
  uint32_t before = 0, higher = 0;
  for (uint32_t i = 0; i < n_mb; ++i) {
    const uint32_t bi = mb_bucket[i];
    const uint64_t ci = mb_cost[i];
    higher += bi > bj;
    before += (bi > bj) || (bi == bj && (ci > cj || (ci == cj && i < j)));
  }
  // index in the bucket's descending list; variant: in the concatenation of all lists (the zig-zag carries on)
  const uint32_t a = carry ? before : before - higher;
  const uint32_t rnd = a / N, i = a % N;
  mb_pos[j] = before;
  mb_rank[j] = (rnd & 1) ? N - 1 - i : i;
}

__global__ void k_rank_index(const uint32_t* mb_pos, const uint32_t* mb_rank, const uint32_t* scalars, uint32_t* mb_idx,
                             uint32_t* rank_cnt) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  const uint32_t n_mb = scalars[SC_NMB];
  if (j >= n_mb) return;
  const uint32_t rj = mb_rank[j], pj = mb_pos[j];
  uint32_t idx = 0;
  for (uint32_t i = 0; i < n_mb; ++i) idx += (mb_rank[i] == rj) && (mb_pos[i] < pj);
  mb_idx[j] = idx;
  atomicAdd(&rank_cnt[rj], 1u);
}

__global__ void __launch_bounds__(1024) k_rank_scan(const uint32_t* rank_cnt, uint32_t N, uint32_t* rank_mb_off) {
  uint64_t carry = 0;
  for (uint32_t base = 0; base < N; base += blockDim.x) {
    const uint32_t r = base + threadIdx.x;
    uint64_t total;
    const uint64_t ex = block_exclusive_scan(r < N ? rank_cnt[r] : 0, &total);
    if (r < N) rank_mb_off[r] = (uint32_t)(carry + ex);
    carry += total;
  }
  if (threadIdx.x == 0) rank_mb_off[N] = (uint32_t)carry;
}

__global__ void k_rank_lists(const uint32_t* mb_rank, const uint32_t* mb_idx, const uint32_t* rank_mb_off,
                             const uint32_t* scalars, uint32_t* rank_mbs) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= scalars[SC_NMB]) return;
  rank_mbs[rank_mb_off[mb_rank[j]] + mb_idx[j]] = j;
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace ft

namespace ft {
constexpr size_t kBestfitSmemLimit = 227 * 1024 - 64;
int32_t plan_device_setup(ft_pool* p) {
  FT_CUDA(cudaFuncSetAttribute(k_bestfit<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBestfitSmemLimit));
  FT_CUDA(cudaFuncSetAttribute(k_bestfit<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBestfitSmemLimit));
  FT_CUDA(cudaFuncSetAttribute(k_bestfit<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBestfitSmemLimit));
  FT_CUDA(cudaFuncSetAttribute(k_bestfit<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBestfitSmemLimit));
  (void)p;
  return FT_OK;
}
}  // namespace ft

using namespace ft;

extern "C" __attribute__((visibility("default"))) int32_t plan_destroy(ft_plan* pl) {
  if (!pl) return FT_ERR_INVALID_ARG;
  if (pl->d_block) {
    ft_pool* p = pl->pool;
    cudaEvent_t ev = nullptr;
    // the block goes back to its pool's cache behind an event on the stream of the plan's last kernel: no
    // synchronisation here, and the next plan takes a block whose event has completed
    if (ft::pool_registry_has(p) && p->plan_cache.size() < 8 && cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess &&
        cudaEventRecord(ev, pl->last_stream) == cudaSuccess) {
      p->plan_cache.push_back({pl->d_block, pl->block_cap, ev});
    } else {
      if (ev) cudaEventDestroy(ev);
      cudaGetLastError();
      cudaDeviceSynchronize();
      cudaFree(pl->d_block);
    }
  }
  delete pl;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t pool_plan_microbatches(ft_pool* p, const uint32_t* slot, uint32_t n, const ft_plan_config* cfg,
                                          ft_plan** out, void* stream) {
  if (!p || !cfg || !out) return FT_ERR_INVALID_ARG;
  p->call_seq++;
  const uint32_t L = cfg->budget_L, K = cfg->n_buckets_K, N = cfg->n_ranks_N;
  if (L == 0 || K == 0 || N == 0) return FT_ERR_INVALID_ARG;
  if (L >= (1u << 20)) return FT_ERR_CAPACITY;  // the bitmap hierarchy covers residuals below 2^20
  {  // the largest possible cost A*L + B*L^2 must fit 64 bits
    const unsigned __int128 mx = (unsigned __int128)cfg->coef_A * L + (unsigned __int128)cfg->coef_B * L * L;
    if (mx >> 64) return FT_ERR_INVALID_ARG;
  }
  if (n && !slot) return FT_ERR_INVALID_ARG;
  const ft_pool_config& c = p->cfg;
  {
    std::vector<uint8_t> seen(c.max_samples, 0);
    for (uint32_t t = 0; t < n; ++t) {
      if (slot[t] >= c.max_samples) return FT_ERR_INVALID_ARG;
      const ft_slot_mirror& s = p->slots[slot[t]];
      if (s.state == FT_SLOT_FREE) return FT_ERR_UNKNOWN_SAMPLE;
      if (seen[slot[t]]) return FT_ERR_INVALID_ARG;
      if (s.state != FT_SLOT_READY && !(cfg->flags & FT_PLAN_ALLOW_UNWRITTEN)) return FT_ERR_NOT_READY;
      if (s.seq_len > L) return FT_ERR_TOO_LONG;
      seen[slot[t]] = 1;
    }
  }
  ft_plan* pl = new ft_plan();
  pl->pool = p; pl->cfg = *cfg; pl->n = n; pl->free_epoch = p->free_epoch;
  pl->slots.assign(slot, slot + n);
  pl->slot_generation.resize(n);
  uint64_t total_tokens = 0;
  for (uint32_t t = 0; t < n; ++t) { pl->slot_generation[t] = p->slots[slot[t]].generation; total_tokens += p->slots[slot[t]].seq_len; }
  if (n == 0) {
    pl->h_mb_sample_off.assign(1, 0); pl->h_mb_row_off.assign(1, 0);
    *out = pl;
    return FT_OK;
  }
  // The plan reads the pool's tables only (lengths and states), never embedding bytes: all of its kernels run on the
  // metadata stream, so a plan requested right after the last producer call is made while that call's copy is still
  // streaming on the caller's stream.  (The row words, filled after the summary has come back, read token ids: that
  // one kernel waits for the latest registration's copy of ids, which precedes the producer call's copy.)
  (void)stream;
  cudaStream_t st = p->meta;
  const uint64_t n_tiles = (total_tokens + 31) / 32 + 1;

  // one device block for every plan array
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t n1 = (size_t)n + 1;
  const size_t o_cost = take(n * 8), o_mbcost = take(n * 8), o_srow = take(n1 * 8), o_mbrow = take(n1 * 8), o_plen = take(n * 8);
  const size_t o_recs = take(n * sizeof(MbRec)), o_head = take(((size_t)L + 1) * 4);
  const size_t o_slots = take(n * 4), o_len = take(n * 4), o_smb = take(n * 4), o_srank = take(n * 4);
  const size_t o_pkt = take(n * 4), o_pklen = take(n * 4), o_pkmb = take(n * 4);
  const size_t o_mboff = take(n1 * 4), o_mbs = take(n * 4), o_psmb = take(n * 4);
  const size_t o_tok = take(n * 4), o_lmax = take(n * 4), o_res = take(n * 4), o_cnt = take(n * 4);
  const size_t o_bkt = take(n * 4), o_rank = take(n * 4), o_pos = take(n * 4), o_idx = take(n * 4);
  const size_t o_roff = take(((size_t)N + 1) * 4), o_rmbs = take(n * 4), o_rcnt = take((size_t)N * 4);
  const size_t o_tiles = take(n_tiles * 4), o_scal = take(SC_COUNT * 4);
  // row words of the assembly: only where every sample is written (a metadata-only plan is not assembled from)
  const bool with_rows = !(cfg->flags & FT_PLAN_ALLOW_UNWRITTEN);
  const size_t o_rows = with_rows ? take((size_t)total_tokens * 8) : 0;
  pl->last_stream = st;
  {
    // a cached block that is large enough: one nobody reads any more if there is one, else the metadata stream
    // waits for its last reader; a fresh allocation only when the cache has none
    int pick = -1;
    for (int i = 0; i < (int)p->plan_cache.size(); ++i) {
      if (p->plan_cache[i].cap < off) continue;
      const bool done = cudaEventQuery(p->plan_cache[i].ev) == cudaSuccess;
      if (done) { pick = i; break; }
      if (pick < 0) pick = i;
    }
    cudaGetLastError();
    if (pick >= 0) {
      ft_pool::plan_block b = p->plan_cache[pick];
      p->plan_cache.erase(p->plan_cache.begin() + pick);
      cudaError_t e = cudaStreamWaitEvent(st, b.ev, 0);
      cudaEventDestroy(b.ev);
      if (e != cudaSuccess) { cudaFree(b.d); delete pl; return ft::cuda_fail(e, "cudaStreamWaitEvent(plan block)"); }
      pl->d_block = b.d; pl->block_cap = b.cap;
    } else {
      if (!p->plan_cache.empty()) {  // only blocks that are too small: let one go, so that the cache cannot clog
        ft_pool::plan_block b = p->plan_cache.front();
        p->plan_cache.erase(p->plan_cache.begin());
        cudaEventSynchronize(b.ev); cudaEventDestroy(b.ev); cudaFree(b.d);
        cudaGetLastError();
      }
      size_t cap = 1 << 20;
      while (cap < off) cap <<= 1;
      cudaError_t e = cudaMalloc(&pl->d_block, cap);
      if (e != cudaSuccess) { delete pl; return ft::cuda_fail(e, "cudaMalloc(plan)"); }
      pl->block_cap = cap;
    }
  }
  uint8_t* b = static_cast<uint8_t*>(pl->d_block);
#define U32(o) reinterpret_cast<uint32_t*>(b + (o))
#define U64(o) reinterpret_cast<uint64_t*>(b + (o))
  pl->d_sample_cost = U64(o_cost); pl->d_mb_cost = U64(o_mbcost); pl->d_sample_row_off = U64(o_srow);
  pl->d_mb_row_off = U64(o_mbrow); pl->d_plan_len = U64(o_plen);
  pl->d_slots = U32(o_slots); pl->d_len = U32(o_len); pl->d_sample_mb = U32(o_smb); pl->d_sample_rank = U32(o_srank);
  pl->d_mb_sample_off = U32(o_mboff); pl->d_mb_samples = U32(o_mbs); pl->d_plan_sample_mb = U32(o_psmb);
  pl->d_mb_tokens = U32(o_tok); pl->d_mb_lmax = U32(o_lmax); pl->d_mb_residual = U32(o_res); pl->d_mb_count = U32(o_cnt);
  pl->d_mb_bucket = U32(o_bkt); pl->d_mb_rank = U32(o_rank); pl->d_mb_pos = U32(o_pos);
  pl->d_rank_mb_off = U32(o_roff); pl->d_rank_mbs = U32(o_rmbs); pl->d_rank_cnt = U32(o_rcnt);
  pl->d_tile_first_sample = U32(o_tiles); pl->d_scalars = U32(o_scal);
  pl->d_row_src = with_rows ? U64(o_rows) : nullptr;
  uint32_t* d_mb_idx = U32(o_idx);
  uint32_t *d_pk_t = U32(o_pkt), *d_pk_len = U32(o_pklen), *d_pk_mb = U32(o_pkmb);
  MbRec* d_recs = reinterpret_cast<MbRec*>(b + o_recs);
  uint32_t* d_head = U32(o_head);

  int32_t rc = FT_OK;
#define CK(call)                                                                            \
  do {                                                                                      \
    cudaError_t e__ = (call);                                                               \
    if (e__ != cudaSuccess) { rc = ft::cuda_fail(e__, #call); plan_destroy(pl); return rc; } \
  } while (0)
  // the slot list goes up through a call context (scratch front), then into the plan
  ft_call_ctx* cx = nullptr;
  rc = ctx_acquire(p, 1, (size_t)n * 4, (size_t)n * 4, &cx);
  if (rc != FT_OK) { plan_destroy(pl); return rc; }
  memcpy(cx->h, slot, (size_t)n * 4);
  rc = ctx_upload(p, cx, (size_t)n * 4);
  if (rc != FT_OK) { plan_destroy(pl); return rc; }
  if ((rc = copy_words(pl->d_slots, cx->d, n, st)) != FT_OK) { plan_destroy(pl); return rc; }
  rc = ctx_release(p, cx, st);
  if (rc != FT_OK) { plan_destroy(pl); return rc; }
  CK(cudaMemsetAsync(pl->d_rank_cnt, 0, (size_t)N * 4, st));

  const unsigned gb = (n + 255) / 256;
  k_plan_prepare<<<gb, 256, 0, st>>>(p->view, pl->d_slots, n, cfg->coef_A, cfg->coef_B, pl->d_len, pl->d_sample_cost);

  // shared memory plan of k_bestfit: bitmaps, staging chunk, then the stack heads and records if they fit
  size_t words = 0;
  { uint32_t w = (L + 1 + 31) / 32; for (int l = 0; l < 4; ++l) { words += w + 1; w = (w + 31) / 32; } }  // one pad word per level
  // (The packing kernel wants most of an SM's storage as shared memory, so it cannot start on an SM that still holds
  // CTAs of a copy kernel with their small shared-memory split; keeping its tables in global memory instead lets it
  // run beside the copies, but every dependent access then pays the loaded memory system's latency: 4.5 ms instead
  // of 0.25 ms for 512 samples.  It therefore keeps its tables in shared memory and runs when an SM is free.)
  const size_t fixed = (words + 3 * (size_t)kFitChunk) * 4 + 16;
  const size_t limit = kBestfitSmemLimit;
  const size_t head_bytes = ((size_t)L + 1) * 4;
  const uint32_t head_in_smem = fixed + head_bytes + 1024 * sizeof(MbRec) <= limit;
  size_t used = fixed + (head_in_smem ? head_bytes : 0);
  const uint32_t rec_cap = (uint32_t)std::min<size_t>(n, (limit - used) / sizeof(MbRec));
  used += (size_t)rec_cap * sizeof(MbRec);
  const uint32_t f_sort = (cfg->flags & FT_PLAN_SORT_DECREASING) != 0, f_sumsq = (cfg->flags & FT_PLAN_COST_SUMSQ) != 0;
  const uint32_t f_carry = (cfg->flags & FT_PLAN_ZIGZAG_CARRY) != 0;
  k_pack_order<<<gb, 256, 0, st>>>(pl->d_len, n, f_sort, d_pk_t, d_pk_len);
  // few microbatches (n_mb <= 2 sum(l)/L + 1 for any-fit packing): the warp-wide kernel; else the bitmap descent
  const uint64_t mb_bound = std::min<uint64_t>(n, 2 * total_tokens / L + 1);
  if (mb_bound <= 128) {
    k_bestfit_regs<4><<<1, 256, 0, st>>>(d_pk_len, n, L, d_pk_mb, pl->d_sample_rank, pl->d_mb_residual, pl->d_mb_tokens, pl->d_mb_lmax,
                                         pl->d_mb_count, pl->d_scalars);
  } else if (mb_bound <= 256) {
    k_bestfit_regs<8><<<1, 256, 0, st>>>(d_pk_len, n, L, d_pk_mb, pl->d_sample_rank, pl->d_mb_residual, pl->d_mb_tokens, pl->d_mb_lmax,
                                         pl->d_mb_count, pl->d_scalars);
  } else if (mb_bound <= kWarpFitMaxCap) {
    const uint32_t cap = (uint32_t)align_up((size_t)mb_bound, 64);
    k_bestfit_warp<<<1, 256, ((size_t)4 * cap + 3 * kWarpFitChunk) * 4, st>>>(d_pk_len, n, L, cap, d_pk_mb, pl->d_sample_rank, pl->d_mb_residual,
                                                                          pl->d_mb_tokens, pl->d_mb_lmax, pl->d_mb_count, pl->d_scalars);
  } else {
    const bool all_recs = rec_cap >= n;
    auto fit = head_in_smem ? (all_recs ? k_bestfit<true, true> : k_bestfit<true, false>)
                            : (all_recs ? k_bestfit<false, true> : k_bestfit<false, false>);
    fit<<<1, n > 8192 ? 1024 : 256, used, st>>>(d_pk_len, n, L, d_head, d_recs, rec_cap, d_pk_mb, pl->d_sample_rank, pl->d_mb_residual,
                               pl->d_mb_tokens, pl->d_mb_lmax, pl->d_mb_count, pl->d_scalars);
  }
  k_mb_finalize<<<1, scan_threads(n), 0, st>>>(pl->d_mb_tokens, pl->d_mb_count, pl->d_mb_sample_off, pl->d_mb_row_off, pl->d_scalars);
  k_plan_scatter<<<gb, 256, 0, st>>>(pl->d_slots, d_pk_t, d_pk_len, d_pk_mb, pl->d_sample_rank, pl->d_mb_sample_off, n,
                                     pl->d_mb_samples, pl->d_plan_len, pl->d_plan_sample_mb, pl->d_sample_mb);
  k_mb_cost<<<gb, 256, 0, st>>>(cfg->coef_A, cfg->coef_B, f_sumsq, pl->d_mb_tokens, pl->d_mb_lmax, pl->d_mb_sample_off,
                                pl->d_plan_len, pl->d_mb_cost, pl->d_scalars);
  k_row_offsets<<<1, scan_threads(n), 0, st>>>(pl->d_plan_len, n, pl->d_sample_row_off);
  k_tiles<<<(unsigned)((n_tiles + 255) / 256), 256, 0, st>>>(pl->d_sample_row_off, n, n_tiles, pl->d_tile_first_sample);
  k_bucket<<<gb, 256, 0, st>>>(pl->d_mb_cost, K, (cfg->flags & FT_PLAN_AUTO_K) ? N : 0u, pl->d_scalars, pl->d_mb_bucket);
  k_sort_deal<<<gb, 256, 0, st>>>(pl->d_mb_cost, pl->d_mb_bucket, N, f_carry, pl->d_scalars, pl->d_mb_pos, pl->d_mb_rank);
  k_rank_index<<<gb, 256, 0, st>>>(pl->d_mb_pos, pl->d_mb_rank, pl->d_scalars, d_mb_idx, pl->d_rank_cnt);
  k_rank_scan<<<1, scan_threads(N), 0, st>>>(pl->d_rank_cnt, N, pl->d_rank_mb_off);
  k_rank_lists<<<gb, 256, 0, st>>>(pl->d_mb_rank, d_mb_idx, pl->d_rank_mb_off, pl->d_scalars, pl->d_rank_mbs);
  CK(cudaGetLastError());
  p->gpu_launches += 13;

  // the summary and the two offset arrays the host sizes assemblies with come back in one go (n + 1 entries bound
  // n_mb + 1), into a pinned landing zone, behind one synchronisation of the metadata stream
  const bool want_copies = with_rows && host_tier_by_copy_engine(p) && p->cfg.host_pages != 0;
  const size_t rb_sc = 0, rb_so = align_up(sizeof(uint32_t) * SC_COUNT, 16), rb_ro = align_up(rb_so + n1 * 4, 16);
  const size_t rb_ms = align_up(rb_ro + n1 * 8, 16), rb_bytes = rb_ms + (want_copies ? (size_t)n * 4 : 0);
  if (p->plan_pinned_cap < rb_bytes) {
    if (p->plan_pinned) CK(cudaFreeHost(p->plan_pinned));
    p->plan_pinned = nullptr; p->plan_pinned_cap = 0;
    size_t cap = 1 << 16;
    while (cap < rb_bytes) cap <<= 1;
    CK(cudaHostAlloc(&p->plan_pinned, cap, cudaHostAllocMapped));
    CK(cudaHostGetDevicePointer(&p->plan_pinned_dev, p->plan_pinned, 0));
    p->plan_pinned_cap = cap;
  }
  uint8_t* rb = static_cast<uint8_t*>(p->plan_pinned);
  {
    uint8_t* rbd = static_cast<uint8_t*>(p->plan_pinned_dev);  // the landing zone as the device sees it
    if ((rc = copy_words(rbd + rb_sc, pl->d_scalars, SC_COUNT, st)) != FT_OK) { plan_destroy(pl); return rc; }
    if ((rc = copy_words(rbd + rb_so, pl->d_mb_sample_off, n1, st)) != FT_OK) { plan_destroy(pl); return rc; }
    if ((rc = copy_words(rbd + rb_ro, pl->d_mb_row_off, n1 * 2, st)) != FT_OK) { plan_destroy(pl); return rc; }
    if (want_copies && (rc = copy_words(rbd + rb_ms, pl->d_mb_samples, n, st)) != FT_OK) { plan_destroy(pl); return rc; }
    p->gpu_launches += want_copies ? 5 : 4;  // these and the copy of the slot list into the plan
  }
  CK(cudaStreamSynchronize(st));
  const uint32_t* sc = reinterpret_cast<const uint32_t*>(rb + rb_sc);
  pl->n_mb = sc[SC_NMB];
  pl->max_mb_tokens = sc[SC_MAXTOK];
  pl->total_tokens = (uint64_t)sc[SC_TOTAL_LO] | ((uint64_t)sc[SC_TOTAL_HI] << 32);
  pl->h_mb_sample_off.assign(reinterpret_cast<const uint32_t*>(rb + rb_so), reinterpret_cast<const uint32_t*>(rb + rb_so) + pl->n_mb + 1);
  pl->h_mb_row_off.assign(reinterpret_cast<const uint64_t*>(rb + rb_ro), reinterpret_cast<const uint64_t*>(rb + rb_ro) + pl->n_mb + 1);
  if (want_copies) {
    // the plan's host-tier pages as copy-engine work, from the host's page lists, in plan order
    const uint32_t* order = reinterpret_cast<const uint32_t*>(rb + rb_ms);
    const uint64_t PS = p->cfg.page_bytes;
    const uint32_t S = p->cfg.max_spans_per_sample;
    const uint8_t* base = static_cast<const uint8_t*>(p->host_base);
    pl->mb_copy_off.assign(pl->n_mb + 1, 0);
    bool ok = true;
    uint64_t row = 0;
    for (uint32_t j = 0; j < pl->n_mb && ok; ++j) {
      for (uint32_t q = pl->h_mb_sample_off[j]; q < pl->h_mb_sample_off[j + 1]; ++q) {
        const uint32_t slot_q = order[q];
        const ft_slot_mirror& sm = p->slots[slot_q];
        if (sm.remote) { ok = false; break; }  // an imported sample: its pages are a peer's, the kernels read them
        for (uint32_t js = 0; js < sm.n_spans; ++js) {
          const ft_span_mirror& m = p->spans[(uint64_t)slot_q * S + js];
          for_each_host_run(p, m, (uint64_t)m.tokens * p->view.row_bytes, [&](uint64_t off, uint64_t frame, uint64_t len) {
            pl->host_copies.push_back({row + m.pos, off, base + frame * PS, len});
          });
        }
        row += sm.seq_len;
      }
      pl->mb_copy_off[j + 1] = (uint32_t)pl->host_copies.size();
    }
    pl->host_copies_valid = ok;
  }
  // the row words are filled behind the caller's back: the plan is complete for the host, assemblies wait for the
  // metadata stream anyway
  rc = plan_rows_launch(p, pl);
  if (rc != FT_OK) { plan_destroy(pl); return rc; }
#undef CK
  *out = pl;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t plan_summary(const ft_plan* pl, uint32_t* n_mb, uint64_t* total_tokens, uint32_t* max_mb_tokens) {
  if (!pl) return FT_ERR_INVALID_ARG;
  if (n_mb) *n_mb = pl->n_mb;
  if (total_tokens) *total_tokens = pl->total_tokens;
  if (max_mb_tokens) *max_mb_tokens = pl->max_mb_tokens;
  return FT_OK;
}

extern "C" __attribute__((visibility("default"))) int32_t plan_arrays(const ft_plan* pl, uint32_t* mb_sample_off, uint32_t* mb_samples, uint32_t* mb_tokens,
                               uint32_t* mb_lmax, uint32_t* mb_residual, uint64_t* mb_cost, uint32_t* mb_bucket,
                               uint32_t* mb_rank, uint32_t* rank_mb_off, uint32_t* rank_mbs, uint64_t* sample_cost,
                               uint32_t* sample_mb) {
  if (!pl) return FT_ERR_INVALID_ARG;
  const size_t n = pl->n, m = pl->n_mb, N = pl->cfg.n_ranks_N;
  if (n == 0) {
    if (mb_sample_off) mb_sample_off[0] = 0;
    if (rank_mb_off) memset(rank_mb_off, 0, (N + 1) * 4);
    return FT_OK;
  }
  FT_CUDA(cudaDeviceSynchronize());
#define CP(dst, src, cnt, sz) \
  if (dst) FT_CUDA(cudaMemcpy(dst, src, (size_t)(cnt) * (sz), cudaMemcpyDeviceToHost))
  CP(mb_sample_off, pl->d_mb_sample_off, m + 1, 4); CP(mb_samples, pl->d_mb_samples, n, 4);
  CP(mb_tokens, pl->d_mb_tokens, m, 4); CP(mb_lmax, pl->d_mb_lmax, m, 4); CP(mb_residual, pl->d_mb_residual, m, 4);
  CP(mb_cost, pl->d_mb_cost, m, 8); CP(mb_bucket, pl->d_mb_bucket, m, 4); CP(mb_rank, pl->d_mb_rank, m, 4);
  CP(rank_mb_off, pl->d_rank_mb_off, N + 1, 4); CP(rank_mbs, pl->d_rank_mbs, m, 4);
  CP(sample_cost, pl->d_sample_cost, n, 8); CP(sample_mb, pl->d_sample_mb, n, 4);
#undef CP
  return FT_OK;
}
