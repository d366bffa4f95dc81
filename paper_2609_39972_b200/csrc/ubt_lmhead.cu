// The step in front of a1, fused with it (Section 3.1.1, eq. 3: the unigram logits of a position are the frozen LM
// head applied to the proposer state): u[row, v] = sum_j hidden[row, j] * weight[v, j], followed directly by the
// vocabulary log-sum-exp and the k best logits of step a1 -- the [rows, V] logits never reach HBM.
//
// One persistent CTA per SM, warp-specialised, on the fifth-generation tensor cores:
//   warp 0  (one lane)  TMA producer: 128 x 64 tiles of hidden and 256 x 64 tiles of weight (bf16, 128-byte
//                       swizzle, no multicast) into a four-stage shared-memory ring
//   warp 1  (one lane)  issues tcgen05.mma (M = 128, N = 256, K = 16, bf16 -> fp32) into one of two 256-column
//                       accumulators in tensor memory; tcgen05.commit frees ring stages and hands accumulators over
//   warps 2-5           epilogue: thread = row of the tile; reads its row of the accumulator with tcgen05.ld,
//                       folds the 256 logits into a running (max, sum exp) and tests them against the row's
//                       exclusive top-k threshold; the few that pass are inserted into the row's sorted list
// A CTA takes vocabulary tiles c, c + grid, ... and, for each, every row tile, so a row's list and (max, sum) are
// carried across all the CTA's vocabulary tiles; one partial per (CTA, row) goes to the workspace and a small
// kernel merges the partials of a row.  The epilogue of one tile runs while the next tile's products accumulate
// in the other half of tensor memory.
//
// Every wait (on a ring stage, on an accumulator) is bounded: a wait that gives up raises a flag, the roles leave
// their loops, the producer waits (bounded again) for the copies still landing, the CTA meets at its last barrier,
// tensor memory is released and the kernel returns; the give-up is counted (ubt_debug_ring_timeouts) and the
// partials of the CTA carry the count -1.
#include <cuda.h>

#include <mutex>

#include "ubt_internal.h"

namespace ubt {

constexpr int LM_BM = 128, LM_BN = 256, LM_BK = 64, LM_STAGES = 4;
constexpr int LM_THREADS = 192;              // warp 0 producer, warp 1 MMA, warps 2-5 epilogue
constexpr int LM_MAX_RT = 16;                // row tiles per launch (2048 rows); more rows take more launches
constexpr int LM_MAX_K = 16;                 // candidates per row the fused epilogue keeps
constexpr int LM_A_BYTES = LM_BM * LM_BK * 2, LM_B_BYTES = LM_BN * LM_BK * 2, LM_STAGE_BYTES = LM_A_BYTES + LM_B_BYTES;
constexpr int LM_SPIN_LIMIT = 1 << 22;

static __device__ unsigned int g_lm_timeouts;

struct LmShared {  // behind the ring in dynamic shared memory
  uint64_t full[LM_STAGES], empty[LM_STAGES], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int fail;
  float m[LM_MAX_RT][LM_BM], s[LM_MAX_RT][LM_BM], thr[LM_MAX_RT][LM_BM];
  unsigned char cnt[LM_MAX_RT][LM_BM];
};

__device__ __forceinline__ uint32_t lm_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void lm_bar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(lm_smem(bar)), "r"(count));
}
__device__ __forceinline__ void lm_bar_expect(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(lm_smem(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void lm_bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(lm_smem(bar)) : "memory");
}
// Bounded wait for the phase with the given parity; false = gave up (counted).
__device__ __forceinline__ bool lm_bar_wait(uint64_t* bar, uint32_t parity, volatile int* fail) {
  for (int spins = 0; spins < LM_SPIN_LIMIT; ++spins) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(lm_smem(bar)), "r"(parity)
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
                   lm_smem(dst)),
               "l"(map), "r"(x), "r"(y), "r"(lm_smem(bar))
               : "memory");
}
// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes under the 128-byte swizzle:
// start address, stride between groups of eight rows (1024 bytes), descriptor version 1, swizzle mode 2.
__device__ __forceinline__ uint64_t lm_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);        // [0,14)  start address >> 4
  d |= (uint64_t)1 << 16;                              // [16,30) leading byte offset >> 4 (unused with this swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                    // [32,46) stride byte offset >> 4
  d |= (uint64_t)1 << 46;                              // [46,48) descriptor version
  d |= (uint64_t)2 << 61;                              // [61,64) 128-byte swizzle
  return d;
}
// Instruction descriptor: fp32 accumulator, bf16 x bf16, both operands K-major, N = 256, M = 128.
constexpr uint32_t kLmIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(LM_BN >> 3) << 17) | ((uint32_t)(LM_BM >> 4) << 24);

__device__ __forceinline__ void lm_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t"
      ".reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t"
      "}\n" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(kLmIdesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void lm_commit(uint64_t* bar) {  // arrives on the barrier when the MMAs issued so far are done
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(lm_smem(bar)) : "memory");
}
__device__ __forceinline__ void lm_tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct LmParts {                   // one partial per (CTA, row of the launch's row block)
  float* ms;                       // [grid, rpad, 2] (max, sum exp relative to it)
  unsigned long long* list;        // [grid, rpad, k] (value, ~token) keys, best first
  int32_t* cnt;                    // [grid, rpad]
  int rpad;                        // rows of the block rounded up to whole row tiles
};

__global__ void __launch_bounds__(LM_THREADS, 1)
k_lm_head_topk(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w, int rows, int d,
               int V, int k, LmParts parts, int* __restrict__ fail_flag) {
  extern __shared__ __align__(1024) unsigned char lm_smem_raw[];
  unsigned char* ring = lm_smem_raw;
  LmShared& sh = *reinterpret_cast<LmShared*>(lm_smem_raw + LM_STAGES * LM_STAGE_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = gridDim.x, cta = blockIdx.x;
  const int n_rt = (rows + LM_BM - 1) / LM_BM, n_vt = (V + LM_BN - 1) / LM_BN, n_kb = d / LM_BK;
  const int my_vt = cta < n_vt ? (n_vt - cta + G - 1) / G : 0;   // vocabulary tiles cta, cta + G, ...
  const int n_items = my_vt * n_rt;
  volatile int* fail = &sh.fail;

  if (tid == 0) {
    for (int s = 0; s < LM_STAGES; ++s) { lm_bar_init(&sh.full[s], 1); lm_bar_init(&sh.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { lm_bar_init(&sh.acc_full[a], 1); lm_bar_init(&sh.acc_empty[a], 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    sh.fail = 0;
  }
  for (int i = tid; i < LM_MAX_RT * LM_BM; i += LM_THREADS) {
    (&sh.m[0][0])[i] = -1.0e30f; (&sh.s[0][0])[i] = 0.f; (&sh.thr[0][0])[i] = -INFINITY; (&sh.cnt[0][0])[i] = 0;
  }
  if (warp == 1) {  // tensor memory: both accumulators (512 columns), allocated by one warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(lm_smem(&sh.tmem_base)), "r"(512u) : "memory");
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
        const int vt = cta + (item / n_rt) * G, rt = item % n_rt;
        for (int kb = 0; kb < n_kb; ++kb, ++it) {
          const int s = it % LM_STAGES;
          const uint32_t ph = (uint32_t)(it / LM_STAGES) & 1u;
          if (!lm_bar_wait(&sh.empty[s], ph ^ 1u, fail)) break;
          lm_bar_expect(&sh.full[s], LM_STAGE_BYTES);
          unsigned char* a = ring + (size_t)s * LM_STAGE_BYTES;
          lm_tma_load(a, &map_h, kb * LM_BK, rt * LM_BM, &sh.full[s]);
          lm_tma_load(a + LM_A_BYTES, &map_w, kb * LM_BK, vt * LM_BN, &sh.full[s]);
        }
      }
      if (*fail)  // gave up: before the CTA leaves, wait (bounded) for the copies still landing in its ring
        for (int i = it > LM_STAGES ? it - LM_STAGES : 0; i < it; ++i)
          lm_bar_wait(&sh.full[i % LM_STAGES], (uint32_t)(i / LM_STAGES) & 1u, fail);
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      int it = 0;
      for (int item = 0; item < n_items && !*fail; ++item) {
        const int ab = item & 1;
        const uint32_t aph = (uint32_t)(item >> 1) & 1u;
        if (!lm_bar_wait(&sh.acc_empty[ab], aph ^ 1u, fail)) break;  // the epilogue has drained this accumulator
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem + (uint32_t)(ab * LM_BN);
        bool ok = true;
        for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
          const int s = it % LM_STAGES;
          const uint32_t ph = (uint32_t)(it / LM_STAGES) & 1u;
          ok = lm_bar_wait(&sh.full[s], ph, fail);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = lm_smem(ring + (size_t)s * LM_STAGE_BYTES), b_addr = a_addr + LM_A_BYTES;
#pragma unroll
          for (int kk = 0; kk < LM_BK / 16; ++kk)  // 16 bf16 = 32 bytes along K inside the swizzled row
            lm_mma(d_tmem, lm_desc(a_addr + kk * 32), lm_desc(b_addr + kk * 32), (kb | kk) != 0 ? 1u : 0u);
          lm_commit(&sh.empty[s]);  // the stage may be refilled once these MMAs have read it
        }
        if (!ok) break;
        lm_commit(&sh.acc_full[ab]);  // the accumulator is complete once every MMA above is
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue: thread = row of the tile
    const int lg = warp & 3;                      // the TMEM lanes this warp may read: 32 * (warp % 4) ...
    const int r_in_tile = lg * 32 + lane;
    for (int item = 0; item < n_items && !*fail; ++item) {
      const int vt = cta + (item / n_rt) * G, rt = item % n_rt;
      const int ab = item & 1;
      const uint32_t aph = (uint32_t)(item >> 1) & 1u;
      if (!lm_bar_wait(&sh.acc_full[ab], aph, fail)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int row = rt * LM_BM + r_in_tile;
      float m = sh.m[rt][r_in_tile], ssum = sh.s[rt][r_in_tile], thr = sh.thr[rt][r_in_tile];
      int cnt = sh.cnt[rt][r_in_tile];
      unsigned long long* list = parts.list + ((size_t)cta * parts.rpad + row) * k;
      const uint32_t taddr = tmem + ((uint32_t)(lg * 32) << 16) + (uint32_t)(ab * LM_BN);
      const int col_base = vt * LM_BN;
#pragma unroll 1
      for (int c0 = 0; c0 < LM_BN; c0 += 32) {
        uint32_t r[32];
        lm_tmem_ld32(taddr + (uint32_t)c0, r);
        const int ncol = V - (col_base + c0);     // columns of this chunk that exist (the last tile is ragged)
        if (ncol <= 0 || row >= rows) continue;   // (every lane still took part in the load above)
        float cm = -INFINITY;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float x = __uint_as_float(r[j]);
          if (j < ncol) cm = fmaxf(cm, x);
        }
        if (cm > m) {  // online log-sum-exp: move the running maximum up
          ssum *= exp2f((m - cm) * kLog2e);
          m = cm;
        }
        const float negm = -m * kLog2e;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float x = __uint_as_float(r[j]);
          if (j < ncol) ssum += exp2f(fmaf(x, kLog2e, negm));
        }
        if (cm > thr || cnt < k) {  // some logit of the chunk enters the row's list
#pragma unroll 1
          for (int j = 0; j < 32 && j < ncol; ++j) {
            const float x = __uint_as_float(r[j]);
            if (!(x > thr) && cnt >= k) continue;   // columns ascend: an equal value loses to the one already kept
            const unsigned long long key = make_key(x, col_base + c0 + j);
            int pos = cnt < k ? cnt : k - 1;        // a full list drops its last entry
            while (pos > 0 && list[pos - 1] < key) { list[pos] = list[pos - 1]; --pos; }
            list[pos] = key;
            cnt = cnt < k ? cnt + 1 : k;
            if (cnt == k) thr = key_val(list[k - 1]);
          }
        }
      }
      if (row < rows) {
        sh.m[rt][r_in_tile] = m; sh.s[rt][r_in_tile] = ssum; sh.thr[rt][r_in_tile] = thr;
        sh.cnt[rt][r_in_tile] = (unsigned char)cnt;
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) lm_bar_arrive(&sh.acc_empty[ab]);  // this warp's quarter of the accumulator is drained
    }
    // partial of every row this thread owns (all row tiles), for the merge
    for (int rt = 0; rt < n_rt; ++rt) {
      const int row = rt * LM_BM + r_in_tile;
      if (row >= rows) continue;
      const size_t slot = (size_t)cta * parts.rpad + row;
      parts.ms[slot * 2] = sh.m[rt][r_in_tile];
      parts.ms[slot * 2 + 1] = sh.s[rt][r_in_tile];
      parts.cnt[slot] = *fail ? -1 : (int)sh.cnt[rt][r_in_tile];
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
k_lm_head_merge(LmParts parts, int grid, int rows, int k, int32_t* __restrict__ cand_ids, float* __restrict__ cand_lp) {
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
      if (lane == 0) { cand_ids[(size_t)row * k + r] = -1; cand_lp[(size_t)row * k + r] = -INFINITY; }
      continue;
    }
    const unsigned holders = __ballot_sync(FULL, best == win);  // keys are unique: one lane holds it
    if (lane == __ffs(holders) - 1) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        if (q == bq) head[q] += 1;
      cand_ids[(size_t)row * k + r] = key_idx(win);
      cand_lp[(size_t)row * k + r] = key_val(win) - lse;
    }
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

size_t lm_head_workspace_bytes(int64_t rows, int k) {
  const size_t grid = (size_t)device_info().sm_count;
  const size_t blk = (size_t)(rows < LM_MAX_RT * LM_BM ? rows : LM_MAX_RT * LM_BM);
  const size_t rpad = (blk + LM_BM - 1) / LM_BM * LM_BM;
  return 256 + lm_align(grid * rpad * 2 * sizeof(float)) + lm_align(grid * rpad * (size_t)k * 8) +
         lm_align(grid * rpad * sizeof(int32_t));
}

// Returns cudaSuccess, or an error; *device_failed (host) is set if a bounded wait gave up on the device.
cudaError_t launch_lm_head_topk(const void* hidden, const void* weight, int64_t rows, int d, int V, int k,
                                int32_t* cand_ids, float* cand_lp, void* ws, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  const int grid = device_info().sm_count;
  const size_t smem = (size_t)LM_STAGES * LM_STAGE_BYTES + sizeof(LmShared);
  cudaError_t e = allow_max_dynamic_smem<k_lm_head_topk>();
  if (e != cudaSuccess) return e;
  unsigned char* p = static_cast<unsigned char*>(ws);
  int* fail_flag = reinterpret_cast<int*>(p); p += 256;
  const int64_t blk_rows = LM_MAX_RT * LM_BM;
  const size_t rpad = (size_t)((rows < blk_rows ? rows : blk_rows) + LM_BM - 1) / LM_BM * LM_BM;
  LmParts parts{};
  parts.rpad = (int)rpad;
  parts.ms = reinterpret_cast<float*>(p); p += lm_align((size_t)grid * rpad * 2 * sizeof(float));
  parts.list = reinterpret_cast<unsigned long long*>(p); p += lm_align((size_t)grid * rpad * (size_t)k * 8);
  parts.cnt = reinterpret_cast<int32_t*>(p);
  e = cudaMemsetAsync(fail_flag, 0, 256, st);
  if (e != cudaSuccess) return e;
  CUtensorMap map_w;
  if (!make_map(&map_w, weight, (uint64_t)d, (uint64_t)V, LM_BN)) return cudaErrorNotSupported;
  for (int64_t r0 = 0; r0 < rows; r0 += blk_rows) {  // blocks of at most 2048 rows (the weight table is re-read per block)
    const int nr = (int)(rows - r0 < blk_rows ? rows - r0 : blk_rows);
    CUtensorMap map_h;
    if (!make_map(&map_h, static_cast<const unsigned char*>(hidden) + (size_t)r0 * d * 2, (uint64_t)d, (uint64_t)nr, LM_BM))
      return cudaErrorNotSupported;
    k_lm_head_topk<<<grid, LM_THREADS, smem, st>>>(map_h, map_w, nr, d, V, k, parts, fail_flag);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    k_lm_head_merge<<<(nr + 3) / 4, 128, 0, st>>>(parts, grid, nr, k, cand_ids + (size_t)r0 * k, cand_lp + (size_t)r0 * k);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t lm_head_timeouts(unsigned int* out) { return cudaMemcpyFromSymbol(out, g_lm_timeouts, sizeof *out); }

}  // namespace ubt
