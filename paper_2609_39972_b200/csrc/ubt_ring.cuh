// Shared-memory ring fed by bulk asynchronous copies (1-D TMA, cp.async.bulk) for the V-wide streaming kernels.
//
// One CTA per SM walks a contiguous span of the flattened [rows, V] logits in chunks that never cross a row.
// An elected thread keeps STAGES-1 chunks in flight; every chunk lands in one stage and completes an
// mbarrier that all threads wait on; the CTA barrier that ends a chunk's processing frees its stage.  The
// copies keep flowing while the CTA is busy, so the bytes in flight per SM do not depend on how the consumer
// code is scheduled.
//
// Every wait is bounded: after kRingSpinLimit failed polls a thread gives up and raises a device-side flag
// (ubt_debug_ring_timeouts); the CTA barrier that ends the chunk carries that vote, so all threads leave the
// loop together, thread 0 waits (again bounded) for the copies still in flight, and the kernel returns.
#pragma once

#include "ubt_common.cuh"

namespace ubt {

constexpr int kRingThreads = 512;
constexpr int kRingSpinLimit = 1 << 20;

static __device__ unsigned int g_ring_timeouts;  // one per translation unit; 0 unless a wait gave up

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// The same poll, but the hardware may keep the thread suspended for up to `hint_ns` while the phase is
// incomplete: a waiting warp then takes (almost) no issue slots from the warps that share its scheduler.
__device__ __forceinline__ bool mbar_try_wait_hint(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_hint(uint64_t* bar, uint32_t parity, uint32_t hint_ns);
// Bounded wait; false = gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (int spins = 0; spins < kRingSpinLimit; ++spins)
    if (mbar_try_wait(bar, parity)) return true;
  atomicAdd(&g_ring_timeouts, 1u);
  return false;
}
__device__ __forceinline__ bool mbar_wait_hint(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
  for (int spins = 0; spins < kRingSpinLimit; ++spins)
    if (mbar_try_wait_hint(bar, parity, hint_ns)) return true;
  atomicAdd(&g_ring_timeouts, 1u);
  return false;
}
// Global -> shared bulk copy; bytes a multiple of 16, both addresses 16-byte aligned.  No multicast.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // earlier generic reads of the stage are done
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(smem_dst)),
               "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}

// The same copy with an L2 eviction priority: a kernel that passes over a row twice asks L2 to let go first of the
// lines its second pass reads (they are not needed again).
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_load_hint(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar,
                                               uint64_t policy) {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // earlier generic reads of the stage are done
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_addr(smem_dst)),
      "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
      : "memory");
}

// Row segment of a CTA's span that starts at flat position `pos`: its row, first column and length.
struct Segment {
  int64_t row;
  int col0, len;
  __device__ __forceinline__ void at(int64_t pos, int64_t hi, int V) {
    row = pos / V;
    col0 = (int)(pos - row * V);
    const int64_t rest = hi - pos;
    len = (int64_t)(V - col0) < rest ? V - col0 : (int)rest;
  }
};

// Consumer-side ring position: stage index and the parity of the phase being waited for.
template <int STAGES>
struct RingPos {
  int stage;
  uint32_t parity;
  __device__ __forceinline__ void init() { stage = 0; parity = 0u; }
  __device__ __forceinline__ void next() {
    if (++stage == STAGES) { stage = 0; parity ^= 1u; }
  }
};

// The producer side: thread 0 of the CTA owns one of these.  It walks the same chunk sequence as the
// consumers (chunks of at most one stage that stop at row ends), STAGES-1 chunks ahead.
template <typename T, int STAGES, int STAGE_BYTES>
struct RingProducer {
  static constexpr int kStageElems = STAGE_BYTES / (int)sizeof(T);
  int64_t pos, hi;
  int V, rem, stage, issued;
  __device__ __forceinline__ void init(int64_t lo, int64_t hi_, int V_) {
    pos = lo; hi = hi_; V = V_; stage = 0; issued = 0;
    Segment sg;
    sg.at(lo, hi_, V_);
    rem = lo < hi_ ? sg.len : 0;
  }
  __device__ __forceinline__ void issue_one(const T* base, unsigned char* ring, uint64_t* full) {
    if (rem == 0) return;
    const int l = rem < kStageElems ? rem : kStageElems;
    mbar_expect_tx(&full[stage], (uint32_t)(l * sizeof(T)));
    bulk_load(ring + (size_t)stage * STAGE_BYTES, base + pos, (uint32_t)(l * sizeof(T)), &full[stage]);
    pos += l;
    rem -= l;
    if (rem == 0 && pos < hi) {
      Segment sg;
      sg.at(pos, hi, V);
      rem = sg.len;
    }
    if (++stage == STAGES) stage = 0;
    ++issued;
  }
  // Advance past one chunk without copying it (for a thread that follows the sequence another one issues).
  __device__ __forceinline__ void skip_one() {
    if (rem == 0) return;
    const int l = rem < kStageElems ? rem : kStageElems;
    pos += l;
    rem -= l;
    if (rem == 0 && pos < hi) {
      Segment sg;
      sg.at(pos, hi, V);
      rem = sg.len;
    }
    if (++stage == STAGES) stage = 0;
    ++issued;
  }
  // After an abandoned loop: chunks [consumed, issued) may still be landing; wait for them, bounded.
  __device__ __forceinline__ void drain(int consumed, uint64_t* full) {
    for (int i = consumed; i < issued; ++i) mbar_wait(&full[i % STAGES], (uint32_t)(i / STAGES) & 1u);
  }
};

}  // namespace ubt
