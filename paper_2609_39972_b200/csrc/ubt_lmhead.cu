// The step in front of a1, fused with it (Section 3.1.1, eq. 3: the unigram logits of a position are the frozen LM
// head applied to the proposer state): u[row, v] = sum_j hidden[row, j] * weight[v, j], followed directly by the
// vocabulary log-sum-exp and the k best logits of step a1 -- the [rows, V] logits never reach HBM.
//
// One persistent CTA per SM, warp-specialised, on the fifth-generation tensor cores:
//   warp 0  (one lane)  TMA producer: a stage of the shared-memory ring holds a 256 x 64 tile of hidden and a
//                       256 x 64 tile of weight (bf16, 128-byte swizzle, no multicast), so every weight tile
//                       serves two accumulators; three stages (four of 128 + 256 rows when there are at most
//                       128 rows in all)
//   warp 1  (one lane)  issues tcgen05.mma (M = 128, N = 256, K = 16, bf16 -> fp32): rows 0-127 of the item
//                       into the first 256 columns of tensor memory, rows 128-255 into the other 256;
//                       tcgen05.commit frees ring stages and hands the accumulators over
//   warps 2-5, 6-9      epilogue of the first / second accumulator: thread = row; reads its row with tcgen05.ld
//                       32 columns at a time, folds them into a running (max, sum exp) and, when the largest of
//                       the 32 beats the row's exclusive top-k threshold (or the list is short), extracts the
//                       qualifying logits best first and inserts them into the row's sorted list
// Work items are (vocabulary tile, block of 256 rows) pairs dealt round-robin to the CTAs; a row's list and
// (max, sum) are carried across all the items a CTA gets for it (parked in the workspace between visits), so one
// partial per (CTA, row) is left for a small kernel that merges the partials of a row.  Tensor memory holds
// exactly one item, so the epilogue is not hidden behind the next item's products: it is kept short instead
// (both accumulators drained at once, one row per thread), while the producer refills the ring.
//
// Every wait (on a ring stage, on an accumulator) is bounded: a wait that gives up raises a flag, the roles leave
// their loops, the producer waits (bounded again) for the copies still landing, the CTA meets at its last barrier,
// tensor memory is released and the kernel returns; the give-up is counted (ubt_debug_ring_timeouts) and the
// partials of the CTA carry the count -1.
#include <cuda.h>

#include <mutex>

#include "ubt_internal.h"
#include "ubt_merge.cuh"
#include "ubt_tc.cuh"

namespace ubt {

constexpr int LM_BM = 128, LM_BN = 256, LM_BK = 64;
constexpr int LM_RB = 2 * LM_BM;             // rows of a work item: two accumulators share every weight tile
constexpr int LM_MAX_STAGES = 4;
constexpr int LM_RING_BYTES = 192 * 1024;    // three stages of 64 KB or four of 48 KB
constexpr int LM_THREADS = 320;              // warp 0 producer, warp 1 MMA, warps 2-5 and 6-9 epilogue
constexpr int LM_MAX_K = 16;                 // candidates per row the fused epilogue keeps
constexpr int LM_MAX_ROWS = 64 * LM_RB;      // rows per call (one bit per row block in a CTA's visited mask)
constexpr int LM_B_BYTES = LM_BN * LM_BK * 2;
constexpr int LM_SPIN_LIMIT = 1 << 22;

static __device__ unsigned int g_lm_timeouts;

struct LmShared {  // behind the ring in dynamic shared memory
  uint64_t full[LM_MAX_STAGES], empty[LM_MAX_STAGES], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int fail;
};

__device__ __forceinline__ void lm_bar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(tc_smem(bar)), "r"(count));
}
__device__ __forceinline__ void lm_bar_expect(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tc_smem(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void lm_bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tc_smem(bar)) : "memory");
}
// Bounded wait for the phase with the given parity; false = gave up (counted).
__device__ __forceinline__ bool lm_bar_wait(uint64_t* bar, uint32_t parity, volatile int* fail) {
  for (int spins = 0; spins < LM_SPIN_LIMIT; ++spins) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(tc_smem(bar)), "r"(parity)
                 : "memory");
    if (ok) return true;
    if ((spins & 1023) == 1023 && *fail) return false;  // another role already gave up
  }
  atomicAdd(&g_lm_timeouts, 1u);
  *fail = 1;
  return false;
}
// 2-D tiled bulk load (TMA) of this GPU's own memory; completes on the mbarrier with its byte count.
__device__ __forceinline__ void lm_tma_load(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                   tc_smem(dst)),
               "l"(map), "r"(x), "r"(y), "r"(tc_smem(bar))
               : "memory");
}

struct LmParts {                   // one partial per (CTA, row of the launch's row block)
  float* ms;                       // [grid, rpad, 2] (max, sum exp relative to it)
  unsigned long long* list;        // [grid, rpad, k] (value, ~token) keys, best first
  int32_t* cnt;                    // [grid, rpad]
  int rpad;                        // rows of the block rounded up to whole row tiles
};

// The row's candidate list lives in registers, best first, 0 = no entry (below every key); only its first k
// entries count.  Every new entry depends on the old list alone, so the KR updates are independent instructions.
template <int KR>
__device__ __forceinline__ void lm_list_insert(unsigned long long (&L)[KR], unsigned long long key) {
#pragma unroll
  for (int i = KR - 1; i > 0; --i) L[i] = key > L[i] ? (key > L[i - 1] ? L[i - 1] : key) : L[i];
  L[0] = key > L[0] ? key : L[0];
}
// (number of entries among the first k, exclusive threshold = value of the k-th entry or -inf)
template <int KR>
__device__ __forceinline__ void lm_list_state(const unsigned long long (&L)[KR], int k, int& cnt, float& thr) {
  unsigned long long kth = 0ull;
  cnt = 0;
#pragma unroll
  for (int i = 0; i < KR; ++i) {
    if (i == k - 1) kth = L[i];
    cnt += (i < k && L[i] != 0ull) ? 1 : 0;
  }
  thr = kth != 0ull ? key_val(kth) : -INFINITY;
}

// How the vocabulary is cut into the tiles of the work items: n1 tiles of bn1 columns, then n2 tiles of bn2.
struct LmTiling {
  int bn1, n1, bn2, n2;
  __host__ __device__ int width(int vt) const { return vt < n1 ? bn1 : bn2; }
  __host__ __device__ int col_base(int vt) const { return vt < n1 ? vt * bn1 : n1 * bn1 + (vt - n1) * bn2; }
};

template <int KR>
__global__ void __launch_bounds__(LM_THREADS, 1)
k_lm_head_topk(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
               const __grid_constant__ CUtensorMap map_w2, int rows, int d, int V, int k, int a_rows, int n_stages,
               LmTiling tl, LmParts parts, int* __restrict__ fail_flag) {
  extern __shared__ __align__(1024) unsigned char lm_smem_raw[];
  unsigned char* ring = lm_smem_raw;
  LmShared& sh = *reinterpret_cast<LmShared*>(lm_smem_raw + LM_RING_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  // The vocabulary is cut into tl.n1 tiles of tl.bn1 columns followed by tl.n2 tiles of tl.bn2 columns (multiples
  // of 16, at most LM_BN), chosen on the host so that the work items fill whole rounds over the CTAs; a stage keeps
  // room for LM_BN weight rows whatever the width is.
  const int n_rb = (rows + LM_RB - 1) / LM_RB, n_vt = tl.n1 + tl.n2, n_kb = d / LM_BK;
  const int a_bytes = a_rows * LM_BK * 2, stage_bytes = a_bytes + LM_B_BYTES;
  // work items: (vocabulary tile, row block) pairs, row block fastest, dealt round-robin: cta, cta + G, ...
  const int n_all = n_vt * n_rb;
  const int n_items = cta < n_all ? (n_all - cta + G - 1) / G : 0;
  volatile int* fail = &sh.fail;

  if (tid == 0) {
    for (int s = 0; s < LM_MAX_STAGES; ++s) { lm_bar_init(&sh.full[s], 1); lm_bar_init(&sh.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { lm_bar_init(&sh.acc_full[a], 1); lm_bar_init(&sh.acc_empty[a], 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    sh.fail = 0;
  }
  if (warp == 1) {  // tensor memory: both accumulators (512 columns), allocated by one warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem(&sh.tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sh.tmem_base;

  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    if (lane == 0) {
      int it = 0;
      for (int item = 0; item < n_items && !*fail; ++item) {
        const int g = cta + item * G, vt = g / n_rb, rb = g % n_rb;
        const bool wide = vt < tl.n1;
        const uint32_t tx_bytes = (uint32_t)(a_bytes + tl.width(vt) * LM_BK * 2);
        const int col_base = tl.col_base(vt);
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % n_stages;
          const uint32_t ph = (uint32_t)(it / n_stages) & 1u;
          if (!lm_bar_wait(&sh.empty[s], ph ^ 1u, fail)) break;
          lm_bar_expect(&sh.full[s], tx_bytes);
          unsigned char* a = ring + (size_t)s * stage_bytes;
          lm_tma_load(a, &map_h, kb * LM_BK, rb * LM_RB, &sh.full[s]);
          lm_tma_load(a + a_bytes, wide ? &map_w : &map_w2, kb * LM_BK, col_base, &sh.full[s]);
        }
      }
      if (*fail)  // gave up: before the CTA leaves, wait (bounded) for the copies still landing in its ring
        for (int i = it > n_stages ? it - n_stages : 0; i < it; ++i)
          lm_bar_wait(&sh.full[i % n_stages], (uint32_t)(i / n_stages) & 1u, fail);
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      int it = 0;
      uint32_t use[2] = {0u, 0u};  // how often each accumulator has been handed over
      for (int item = 0; item < n_items && !*fail; ++item) {
        const int rb = (cta + item * G) % n_rb;
        const uint32_t idesc = tc_idesc_bf16(LM_BM, tl.width((cta + item * G) / n_rb));
        const int n_half = rows - rb * LM_RB > LM_BM ? 2 : 1;  // a row block of at most 128 rows fills one accumulator
        bool ok = true;
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int s = it % n_stages;
          const uint32_t ph = (uint32_t)(it / n_stages) & 1u;
          ok = lm_bar_wait(&sh.full[s], ph, fail);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = tc_smem(ring + (size_t)s * stage_bytes), b_addr = a_addr + (uint32_t)a_bytes;
#pragma unroll
          for (int half = 0; half < 2; ++half) {  // rows 0-127 -> accumulator 0, rows 128-255 -> accumulator 1
            if (half >= n_half) break;
            if (kb == 0) {  // the epilogue has drained this accumulator
              ok = lm_bar_wait(&sh.acc_empty[half], (use[half] & 1u) ^ 1u, fail);
              if (!ok) break;
              asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            }
            const uint32_t d_tmem = tmem + (uint32_t)(half * LM_BN);
            const uint32_t ah = a_addr + (uint32_t)(half * LM_BM * LM_BK * 2);
#pragma unroll
            for (int kk = 0; kk < LM_BK / 16; ++kk)  // 16 bf16 = 32 bytes along K inside the swizzled row
              tc_mma(d_tmem, tc_desc(ah + kk * 32), tc_desc(b_addr + kk * 32), idesc, (kb | kk) != 0 ? 1u : 0u);
          }
          if (!ok) break;
          tc_commit(&sh.empty[s]);  // the stage may be refilled once these MMAs have read it
        }
        if (!ok) break;
        for (int half = 0; half < n_half; ++half) {  // complete once every MMA above is
          tc_commit(&sh.acc_full[half]);
          use[half] += 1u;
        }
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue: thread = row of one accumulator
    const int half = (warp - 2) >> 2;
    const int lg = warp & 3;                      // the TMEM lanes this warp may read: 32 * (warp % 4) ...
    const int r_in_tile = lg * 32 + lane;
    const uint32_t taddr = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(half * LM_BN);
    unsigned long long visited = 0ull;            // row blocks this CTA has a partial for already
    uint32_t use = 0u;
    bool ok = true;
    for (int item = 0; item < n_items && !*fail; ++item) {
      const int g = cta + item * G, vt = g / n_rb, rb = g % n_rb;
      if (half == 1 && rows - rb * LM_RB <= LM_BM) continue;  // this item leaves the second accumulator unused
      const uint32_t aph = use & 1u;
      use += 1u;
      const bool first = !((visited >> rb) & 1ull);
      visited |= 1ull << rb;
      const int col_base = tl.col_base(vt), bn = tl.width(vt);
      const int row = rb * LM_RB + half * LM_BM + r_in_tile;
      const bool valid = row < rows;
      const size_t slot = (size_t)cta * parts.rpad + row;
      // the row's running state: from the workspace unless this is the CTA's first visit of the row block
      float m = -1.0e30f, ssum = 0.f, thr;
      int cnt = 0;
      unsigned long long L[KR];
      if (!first && valid) { m = parts.ms[slot * 2]; ssum = parts.ms[slot * 2 + 1]; cnt = parts.cnt[slot]; }
#pragma unroll
      for (int i = 0; i < KR; ++i) L[i] = i < cnt ? parts.list[slot * k + i] : 0ull;
      lm_list_state(L, k, cnt, thr);
      ok = lm_bar_wait(&sh.acc_full[half], aph, fail);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int c0 = 0; c0 < bn; c0 += 32) {
        uint32_t r[32];
        tc_tmem_ld32(taddr + (uint32_t)c0, r);
        // columns of this chunk that belong to the item and exist (the last tile of the vocabulary is ragged)
        const int ncol = min(V - (col_base + c0), bn - c0);
        if (ncol <= 0 || !valid) continue;        // (every lane still took part in the load above)
        if (ncol < 32) {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (j >= ncol) r[j] = 0xff800000u;    // -inf: adds nothing to the sum, never chosen
        }
        float cm = __uint_as_float(r[0]);
#pragma unroll
        for (int j = 1; j < 32; ++j) cm = fmaxf(cm, __uint_as_float(r[j]));
        if (cm > m) {  // online log-sum-exp: move the running maximum up
          ssum *= ex2_approx((m - cm) * kLog2e);
          m = cm;
        }
        const float negm = -m * kLog2e;
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          s0 += ex2_approx(fmaf(__uint_as_float(r[j]), kLog2e, negm));
          s1 += ex2_approx(fmaf(__uint_as_float(r[j + 1]), kLog2e, negm));
        }
        ssum += s0 + s1;
        if (cm > thr || cnt < k) {  // some logit of the chunk enters the row's list
          uint32_t avail = ncol < 32 ? (1u << ncol) - 1u : 0xffffffffu;
          while (cnt < k && avail) {  // a short list (the CTA's first columns of the row): fill it best first
            float best = -INFINITY;
            int bj = -1;
#pragma unroll
            for (int j = 31; j >= 0; --j) {  // ">=" on the way down: of equal values the lowest column wins
              const float x = __uint_as_float(r[j]);
              if (((avail >> j) & 1u) && x >= best) { best = x; bj = j; }
            }
            if (bj < 0) break;
            lm_list_insert(L, make_key(best, col_base + c0 + bj));
            cnt += 1;
            avail &= ~(1u << bj);
          }
          lm_list_state(L, k, cnt, thr);
          // a full list: the columns above the threshold, in ascending order (an equal value loses to the one
          // already kept: columns ascend over a CTA's visits of a row, and within this loop)
          uint32_t q = 0u;
#pragma unroll
          for (int j = 0; j < 32; ++j) q |= (__uint_as_float(r[j]) > thr ? 1u : 0u) << j;
          q &= avail;
          while (q) {
            const int j = __ffs((int)q) - 1;
            q &= q - 1u;
            uint32_t t16[16], t8[8], t4[4], t2[2];  // r[j] by a tree of selects (the registers cannot be indexed)
#pragma unroll
            for (int i = 0; i < 16; ++i) t16[i] = (j & 1) ? r[2 * i + 1] : r[2 * i];
#pragma unroll
            for (int i = 0; i < 8; ++i) t8[i] = (j & 2) ? t16[2 * i + 1] : t16[2 * i];
#pragma unroll
            for (int i = 0; i < 4; ++i) t4[i] = (j & 4) ? t8[2 * i + 1] : t8[2 * i];
#pragma unroll
            for (int i = 0; i < 2; ++i) t2[i] = (j & 8) ? t4[2 * i + 1] : t4[2 * i];
            const float x = __uint_as_float((j & 16) ? t2[1] : t2[0]);
            if (x > thr) {
              lm_list_insert(L, make_key(x, col_base + c0 + j));
              lm_list_state(L, k, cnt, thr);
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) lm_bar_arrive(&sh.acc_empty[half]);  // this warp's quarter of the accumulator is drained
      if (valid) {  // the row's state goes back to the workspace (the merge reads it from there, too)
        parts.ms[slot * 2] = m; parts.ms[slot * 2 + 1] = ssum; parts.cnt[slot] = cnt;
#pragma unroll
        for (int i = 0; i < KR; ++i)
          if (i < cnt) parts.list[slot * k + i] = L[i];
      }
    }
    // rows this CTA never visited (more CTAs than work items) and, after a give-up, every row: empty / marked
    for (int rb = 0; rb < n_rb; ++rb) {
      const bool seen = (visited >> rb) & 1ull;
      if (seen && !*fail) continue;
      const int row = rb * LM_RB + half * LM_BM + r_in_tile;
      if (row >= rows) continue;
      const size_t slot = (size_t)cta * parts.rpad + row;
      if (!seen) { parts.ms[slot * 2] = -1.0e30f; parts.ms[slot * 2 + 1] = 0.f; }
      parts.cnt[slot] = *fail ? -1 : 0;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  if (tid == 0 && *fail) atomicExch(fail_flag, 1);
}

// One warp per row: (max, sum) over the CTAs' partials, then the k best of their sorted lists by k rounds of
// "best head"; cand_lp = value - log-sum-exp.
__global__ void __launch_bounds__(128)
k_lm_head_merge(LmParts parts, int grid, int rows, int k, int32_t* __restrict__ cand_ids, float* __restrict__ cand_lp,
                MergeShardOut so) {
  // so.ms set: this GPU holds a slice of the vocabulary; the row's result is written as the rank's partial of a
  // vocabulary-parallel a1 (raw values, ids moved by the slice's first column, (max, sum exp), count) instead
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  float M = -1.0e30f;
  for (int g = lane; g < grid; g += 32) {
    const size_t slot = (size_t)g * parts.rpad + row;
    if (parts.cnt[slot] > 0 || parts.ms[slot * 2 + 1] > 0.f) M = fmaxf(M, parts.ms[slot * 2]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(FULL, M, o));
  float S = 0.f;
  for (int g = lane; g < grid; g += 32) {
    const size_t slot = (size_t)g * parts.rpad + row;
    S += parts.ms[slot * 2 + 1] * exp2f((parts.ms[slot * 2] - M) * kLog2e);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(FULL, S, o);
  const float lse = M + logf(S);
  // heads: lane owns the lists of CTAs lane, lane + 32, ...; at most 8 lists per lane (grid <= 256)
  int head[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) head[q] = 0;
  int found = 0;
  for (int r = 0; r < k; ++r) {
    unsigned long long best = 0ull;
    int bq = -1;
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int g = lane + 32 * q;
      if (g >= grid) continue;
      const size_t slot = (size_t)g * parts.rpad + row;
      const int c = parts.cnt[slot];
      if (head[q] < c) {
        const unsigned long long key = parts.list[slot * k + head[q]];
        if (key > best) { best = key; bq = q; }
      }
    }
    const unsigned long long win = warp_max_u64(best);
    if (win == 0ull) {  // fewer than k entries in the whole row
      if (lane == 0 && !so.ms) { cand_ids[(size_t)row * k + r] = -1; cand_lp[(size_t)row * k + r] = -INFINITY; }
      continue;
    }
    ++found;
    const unsigned holders = __ballot_sync(FULL, best == win);  // keys are unique: one lane holds it
    if (lane == __ffs(holders) - 1) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (q == bq) head[q] += 1;
      if (so.ms) {
        so.idx[(size_t)row * k + r] = key_idx(win) + so.id_offset;
        so.val[(size_t)row * k + r] = key_val(win);
      } else {
        cand_ids[(size_t)row * k + r] = key_idx(win);
        cand_lp[(size_t)row * k + r] = key_val(win) - lse;
      }
    }
  }
  if (so.ms && lane == 0) {
    so.ms[(size_t)row * 2] = M;
    so.ms[(size_t)row * 2 + 1] = S;
    so.cnt[row] = found;
  }
}

// ------------------------------------------------------------------------------------ host side
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// [outer, inner] bf16 row-major matrix, boxes of box_outer x 64 elements, 128-byte swizzle, zero fill outside.
bool make_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint32_t box_outer) {
  EncodeTiledFn fn = encode_tiled();
  if (!fn) return false;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {inner * 2};
  const cuuint32_t box[2] = {(cuuint32_t)LM_BK, box_outer};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
size_t lm_align(size_t x) { return (x + 255) / 256 * 256; }
}  // namespace

int lm_head_max_k() { return LM_MAX_K; }

int lm_head_max_rows() { return LM_MAX_ROWS; }

size_t lm_head_workspace_bytes(int64_t rows, int k) {
  const size_t grid = (size_t)device_info().sm_count;
  const size_t rpad = ((size_t)rows + LM_RB - 1) / LM_RB * LM_RB;
  return 256 + lm_align(grid * rpad * 2 * sizeof(float)) + lm_align(grid * rpad * (size_t)k * 8) +
         lm_align(grid * rpad * sizeof(int32_t));
}

// Returns cudaSuccess, or an error; *device_failed (host) is set if a bounded wait gave up on the device.
cudaError_t launch_lm_head_topk(const void* hidden, const void* weight, int64_t rows, int d, int V, int k,
                                int32_t* cand_ids, float* cand_lp, void* ws, cudaStream_t st, void* shard_partial,
                                int v0) {
  if (rows == 0) return cudaSuccess;
  const int grid = device_info().sm_count;
  const size_t smem = (size_t)LM_RING_BYTES + sizeof(LmShared);
  const int a_rows = rows <= LM_BM ? LM_BM : LM_RB, n_stages = rows <= LM_BM ? 4 : 3;
  // Width of a work item along the vocabulary: the widest tile is the most efficient one, but the items are dealt
  // in whole rounds over the CTAs, and 594 tiles of 256 columns over 148 CTAs is four rounds and a fifth for two
  // CTAs.  Take the width (a multiple of 16) with the shortest schedule: rounds x (width + the fixed cost of an
  // item in columns' worth).  Measured at d = 4096: an item takes 10 us + 0.17 us per column when one block of
  // rows streams the weights (bound by their bandwidth), and 27 us + 0.12 us per column with two accumulators.
  const int n_rb = (int)((rows + LM_RB - 1) / LM_RB);
  const int fixed_cols = rows <= LM_RB ? 60 : 224;
  LmTiling tl{LM_BN, (V + LM_BN - 1) / LM_BN, LM_BN, 0};
  long long best_cost = -1;
  for (int w = LM_BN; w >= 128; w -= 16) {
    const long long items = (long long)((V + w - 1) / w) * n_rb;
    const long long cost = ((items + grid - 1) / grid) * (w + fixed_cols);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; tl = LmTiling{w, (V + w - 1) / w, w, 0}; }
  }
  // Two widths 16 apart let the number of tiles be chosen freely, so that the items are exactly `rounds` per CTA:
  // 666 tiles of 240 and 224 columns are nine full rounds for two row blocks over 148 CTAs, against nine rounds
  // (the last nearly empty) of 256-column tiles.
  for (long long rounds = 1; rounds <= 4096; ++rounds) {
    const long long n_tiles = rounds * grid / n_rb;
    if (n_tiles < 1 || n_tiles * LM_BN < V) continue;
    const int lo = (int)(V / n_tiles) / 16 * 16;  // the narrower width
    if (lo < 128) break;                          // narrower tiles than the uniform search considers
    const int hi = lo + 16 <= LM_BN ? lo + 16 : LM_BN;
    const long long n_hi = hi > lo ? (V - n_tiles * lo + 15) / 16 : 0;  // tiles that must be 16 columns wider
    if (n_hi > n_tiles) continue;
    const long long cost = rounds * (long long)((V + n_tiles - 1) / n_tiles + fixed_cols);
    if (cost < best_cost) {
      best_cost = cost;
      tl = n_hi > 0 ? LmTiling{hi, (int)n_hi, lo, (int)(n_tiles - n_hi)} : LmTiling{lo, (int)n_tiles, lo, 0};
    }
    break;  // more rounds of narrower tiles only cost more
  }
  cudaError_t e = allow_max_dynamic_smem<k_lm_head_topk<4>>();
  if (e == cudaSuccess) e = allow_max_dynamic_smem<k_lm_head_topk<8>>();
  if (e == cudaSuccess) e = allow_max_dynamic_smem<k_lm_head_topk<16>>();
  if (e != cudaSuccess) return e;
  unsigned char* p = static_cast<unsigned char*>(ws);
  int* fail_flag = reinterpret_cast<int*>(p); p += 256;
  const size_t rpad = ((size_t)rows + LM_RB - 1) / LM_RB * LM_RB;
  LmParts parts{};
  parts.rpad = (int)rpad;
  parts.ms = reinterpret_cast<float*>(p); p += lm_align((size_t)grid * rpad * 2 * sizeof(float));
  parts.list = reinterpret_cast<unsigned long long*>(p); p += lm_align((size_t)grid * rpad * (size_t)k * 8);
  parts.cnt = reinterpret_cast<int32_t*>(p);
  e = cudaMemsetAsync(fail_flag, 0, 256, st);
  if (e != cudaSuccess) return e;
  CUtensorMap map_w, map_w2, map_h;
  if (!make_map(&map_w, weight, (uint64_t)d, (uint64_t)V, (uint32_t)tl.bn1)) return cudaErrorNotSupported;
  if (!make_map(&map_w2, weight, (uint64_t)d, (uint64_t)V, (uint32_t)tl.bn2)) return cudaErrorNotSupported;
  if (!make_map(&map_h, hidden, (uint64_t)d, (uint64_t)rows, (uint32_t)a_rows)) return cudaErrorNotSupported;
  if (k <= 4)
    k_lm_head_topk<4><<<grid, LM_THREADS, smem, st>>>(map_h, map_w, map_w2, (int)rows, d, V, k, a_rows, n_stages, tl, parts, fail_flag);
  else if (k <= 8)
    k_lm_head_topk<8><<<grid, LM_THREADS, smem, st>>>(map_h, map_w, map_w2, (int)rows, d, V, k, a_rows, n_stages, tl, parts, fail_flag);
  else
    k_lm_head_topk<16><<<grid, LM_THREADS, smem, st>>>(map_h, map_w, map_w2, (int)rows, d, V, k, a_rows, n_stages, tl, parts, fail_flag);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  MergeShardOut so{};
  if (shard_partial) so = carve_shard_partial(shard_partial, rows, k, v0);
  k_lm_head_merge<<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(parts, grid, (int)rows, k, cand_ids, cand_lp, so);
  return cudaGetLastError();
}

cudaError_t lm_head_timeouts(unsigned int* out) { return cudaMemcpyFromSymbol(out, g_lm_timeouts, sizeof *out); }

}  // namespace ubt
