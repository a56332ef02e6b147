// Bulk asynchronous copies (the TMA unit's non-tensor form, cp.async.bulk) driven by one warp through a ring
// of shared-memory stages: global -> shared (completion on an mbarrier), then shared -> global (bulk groups).
// One thread keeps `kDepth` loads in flight, so a handful of single-warp CTAs saturate a long-latency link
// (mapped pinned host memory) without tying up the load/store pipelines of the SMs that stream HBM.
// Every copy lands in the issuing CTA only.  Every wait is bounded.
//
// Giving up.  A staged load that has not arrived after the wait limit (2 s unless the pool's tuning says otherwise)
// is declared lost: the ring issues no further load or store, and before the CTA returns drain() waits once more, again bounded, for every load it had already
// issued, so that none of them can land later in shared memory that by then belongs to another CTA; `stranded`
// counts the loads that had still not arrived when that second wait ran out as well (the kernel reports it in the
// error detail).  Stores already issued are waited for with the hardware's group wait.
#pragma once
#include <stdint.h>

namespace ft {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t n) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(n));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(void* dst_s, const void* src_g, uint32_t bytes, uint64_t* b) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst_s)), "l"(src_g), "r"(bytes), "r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* dst_g, const void* src_s, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(dst_g), "r"(smem_u32(src_s)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

constexpr int kBulkStages = 12;            // ring size
constexpr int kBulkDepth = 8;              // loads in flight
constexpr uint32_t kBulkStageBytes = 16384;
constexpr uint64_t kBulkWaitLimitNs = 2000000000ull;  // default: a staged load not seen after 2 s is declared lost
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Warp-wide copy pipeline: every lane of a one-warp CTA calls push()/drain() with the same arguments; lane 0
// issues the asynchronous operations.  Copy number i goes into stage i % kBulkStages; before that, copy
// i - kBulkDepth is retired (wait for its load, start its store).  A stage is reused only after the store
// that last read it has finished reading shared memory.
struct BulkRing {
  uint8_t* stage;    // kBulkStages * kBulkStageBytes of shared memory, 128-byte aligned
  uint64_t* bar;     // kBulkStages mbarriers
  uint64_t* dst_q;   // kBulkStages pending destinations (shared memory)
  uint32_t* len_q;   // kBulkStages pending staged lengths
  uint64_t issued, retired;
  uint64_t limit_ns;  // bound of every wait
  uint32_t tx_slack;  // bytes announced to the barrier beyond the load's size (0; 16 under the timeout test)
  uint32_t stranded;  // loads still not arrived when a CTA that gave up returned
  bool lost;

  __device__ void init(uint8_t* stage_, uint64_t* bar_, uint64_t* dst_q_, uint32_t* len_q_, uint64_t limit_ns_, uint32_t tx_slack_) {
    stage = stage_; bar = bar_; dst_q = dst_q_; len_q = len_q_;
    limit_ns = limit_ns_; tx_slack = tx_slack_;
    issued = retired = 0; lost = false; stranded = 0;
    if ((threadIdx.x & 31) == 0) {
      for (int i = 0; i < kBulkStages; ++i) mbar_init(&bar[i], 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      fence_async_smem();
    }
    __syncwarp();
  }
  __device__ void retire_one() {
    const uint32_t lane = threadIdx.x & 31;
    const uint64_t k = retired++;
    const int st = (int)(k % kBulkStages);
    const uint32_t parity = (uint32_t)((k / kBulkStages) & 1);
    uint32_t bad = 0;
    if (lane == 0 && !mbar_try_wait(&bar[st], parity)) {
      // bounded wait: poll, looking at the wall clock every 1024 polls
      const uint64_t t0 = global_timer_ns();
      uint32_t spins = 0;
      while (!mbar_try_wait(&bar[st], parity)) {
        if ((++spins & 1023u) == 0 && global_timer_ns() - t0 > limit_ns) { bad = 1; break; }
      }
    }
    bad = __shfl_sync(0xFFFFFFFFu, bad, 0);
    if (bad) { lost = true; return; }
    uint8_t* sp = stage + (size_t)st * kBulkStageBytes;
    const uint32_t len = len_q[st];
    if (lane == 0) {
      bulk_s2g(reinterpret_cast<void*>(dst_q[st]), sp, len);
      bulk_commit();
    }
  }
  // bytes: multiple of 16, <= kBulkStageBytes; src and dst 16-byte aligned
  __device__ void push(const void* src, void* dst, uint32_t bytes) {
    if (lost) return;
    if (issued - retired >= (uint64_t)kBulkDepth) retire_one();
    if (lost) return;
    const int st = (int)(issued % kBulkStages);
    if ((threadIdx.x & 31) == 0) {
      bulk_wait_read<kBulkStages - kBulkDepth>();
      dst_q[st] = reinterpret_cast<uint64_t>(dst);
      len_q[st] = bytes;
      mbar_expect_tx(&bar[st], bytes + tx_slack);
      bulk_g2s(stage + (size_t)st * kBulkStageBytes, src, bytes, &bar[st]);
    }
    __syncwarp();
    ++issued;
  }
  __device__ void drain() {
    while (!lost && retired < issued) retire_one();
    if (lost) {
      // gave up: the loads issued before that are still owed to this CTA's shared memory; wait for them, bounded
      uint32_t left = 0;
      if ((threadIdx.x & 31) == 0) {
        const uint64_t t0 = global_timer_ns();
        for (uint64_t k = retired - 1; k < issued; ++k) {  // retired - 1 is the load whose wait ran out
          const int st = (int)(k % kBulkStages);
          const uint32_t parity = (uint32_t)((k / kBulkStages) & 1);
          bool here = mbar_try_wait(&bar[st], parity);
          uint32_t spins = 0;
          while (!here && !((++spins & 1023u) == 0 && global_timer_ns() - t0 > limit_ns)) here = mbar_try_wait(&bar[st], parity);
          if (!here) ++left;
        }
      }
      stranded = __shfl_sync(0xFFFFFFFFu, left, 0);
    }
    if ((threadIdx.x & 31) == 0) bulk_wait_all<0>();
    __syncwarp();
  }
};

constexpr size_t kBulkSmemBytes = (size_t)kBulkStages * kBulkStageBytes;

}  // namespace ft
