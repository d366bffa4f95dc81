// Selector scores of all candidate pairs (Section 3.1.2, "Parallel Computation"):
//   delta_i(a, b) = sum_r g_i[r] * phi[a][r] * psi[b][r],   Delta_i = Phi_{i-1} diag(P(h_i)) Psi_i^T.
//
// One CTA of 256 threads per (sequence, position): a k x k x R product in fp32.  The rank dimension is walked in
// chunks of 256: the k predecessor rows of phi (scaled by the position's gate) and the k successor rows of psi
// are staged in shared memory as fp32, rows padded by four floats so that 16-byte loads of different rows fall
// into different banks; a thread owns the outputs (ty + 16 m, tx + 16 n), m, n < 4, and accumulates them with
// 16-byte shared-memory loads (8 loads feed 64 multiply-adds).  The sum over r runs in index order.
// Work per batch: a gather of 2k table rows per position (a few MB) and B L k^2 R multiply-adds (1 GFLOP for
// B = 32, L = 15, k = 64, R = 256): the kernel is bound by shared-memory bandwidth and launch latency, far from
// HBM and from the fp32 peak.
#include <cuda_bf16.h>

#include "ubt_internal.h"
#include "ubt_tc.cuh"

namespace ubt {

constexpr int GS_T = 256;
constexpr int GS_RC = 256;        // rank elements per chunk
constexpr int GS_LD = GS_RC + 4;  // padded row length in shared memory
constexpr int GS_K = 64;          // rows per operand (kMaxK)

template <typename T>
__global__ void __launch_bounds__(GS_T)
k_selector_scores(const T* __restrict__ phi, const T* __restrict__ psi, int V, int R,
                  const float* __restrict__ gate, const int32_t* __restrict__ cand_ids,
                  const int32_t* __restrict__ anchor_tokens, int L, int k, float* __restrict__ bigram,
                  float* __restrict__ anchor_bigram) {
  extern __shared__ __align__(16) float smem[];
  float* As = smem;                 // [GS_K][GS_LD]  gate[r] * phi[pred[ra]][r]
  float* Bs = smem + GS_K * GS_LD;  // [GS_K][GS_LD]  psi[succ[rb]][r]
  __shared__ int s_pred[GS_K], s_succ[GS_K];
  const int b = blockIdx.x / L, i = blockIdx.x % L;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  if (i == 0 && (anchor_tokens == nullptr || anchor_bigram == nullptr)) return;
  const int npred = i == 0 ? 1 : k;
  if (tid < GS_K) {
    int a = -1, t = -1;
    if (tid < npred) a = i == 0 ? anchor_tokens[b] : cand_ids[((int64_t)b * L + i - 1) * k + tid];
    if (tid < k) t = cand_ids[((int64_t)b * L + i) * k + tid];
    // memory-safe for ids outside the vocabulary; -1 marks a row that does not exist
    s_pred[tid] = tid < npred ? (a < 0 ? 0 : (a >= V ? V - 1 : a)) : -1;
    s_succ[tid] = tid < k ? (t < 0 ? 0 : (t >= V ? V - 1 : t)) : -1;
  }
  __syncthreads();
  const float* g = gate + ((int64_t)b * L + i) * R;
  float acc[4][4];
#pragma unroll
  for (int m = 0; m < 4; ++m)
#pragma unroll
    for (int n = 0; n < 4; ++n) acc[m][n] = 0.f;

  for (int r0 = 0; r0 < R; r0 += GS_RC) {
    const int rc = R - r0 < GS_RC ? R - r0 : GS_RC;
    // stage the chunk: a warp fetches whole table rows, 16 bytes per lane (independent loads, eight rows in
    // flight per warp), widens them to fp32 and scales the phi rows by the gate
    constexpr int VEC = 16 / (int)sizeof(T);        // elements per 16-byte load
    constexpr int LPR = GS_RC / VEC / 32;           // loads per lane and row: 1 (bf16) or 2 (fp32)
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int half = 0; half < 2; ++half) {          // rows [0, 64): phi operand, rows [64, 128): psi operand
      uint4 raw[8][LPR];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int row = warp * 8 + q;               // 8 warps x 8 rows
        const int tok = half == 0 ? s_pred[row] : s_succ[row];
        const T* base = (half == 0 ? phi : psi) + (int64_t)(tok < 0 ? 0 : tok) * R + r0;
#pragma unroll
        for (int h = 0; h < LPR; ++h) {
          const int r = (h * 32 + lane) * VEC;
          raw[q][h] = (tok >= 0 && r < rc) ? __ldg(reinterpret_cast<const uint4*>(base + r)) : make_uint4(0u, 0u, 0u, 0u);
        }
      }
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int row = warp * 8 + q;
        float* dst = (half == 0 ? As : Bs) + row * GS_LD;
#pragma unroll
        for (int h = 0; h < LPR; ++h) {
          const int r = (h * 32 + lane) * VEC;
          Frag<T> fr;
          fr.unpack(raw[q][h]);
#pragma unroll
          for (int j = 0; j < VEC; j += 4) {
            float4 o = make_float4(fr.x[j], fr.x[j + 1], fr.x[j + 2], fr.x[j + 3]);
            if (half == 0) {
              const float4 gv = r + j < rc ? *reinterpret_cast<const float4*>(g + r0 + r + j) : make_float4(0.f, 0.f, 0.f, 0.f);
              o.x *= gv.x; o.y *= gv.y; o.z *= gv.z; o.w *= gv.w;
            }
            *reinterpret_cast<float4*>(dst + r + j) = o;
          }
        }
      }
    }
    __syncthreads();
    const int r4n = (rc + 3) / 4;
    for (int r4 = 0; r4 < r4n; ++r4) {
      float4 av[4], bv[4];
#pragma unroll
      for (int m = 0; m < 4; ++m) av[m] = *reinterpret_cast<const float4*>(As + (ty + 16 * m) * GS_LD + 4 * r4);
#pragma unroll
      for (int n = 0; n < 4; ++n) bv[n] = *reinterpret_cast<const float4*>(Bs + (tx + 16 * n) * GS_LD + 4 * r4);
#pragma unroll
      for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int n = 0; n < 4; ++n) {
          acc[m][n] = fmaf(av[m].x, bv[n].x, acc[m][n]);
          acc[m][n] = fmaf(av[m].y, bv[n].y, acc[m][n]);
          acc[m][n] = fmaf(av[m].z, bv[n].z, acc[m][n]);
          acc[m][n] = fmaf(av[m].w, bv[n].w, acc[m][n]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    const int ra = ty + 16 * m;
    if (ra >= npred) continue;
    float* out = i == 0 ? anchor_bigram + (int64_t)b * k : bigram + (((int64_t)b * (L - 1) + i - 1) * k + ra) * k;
#pragma unroll
    for (int n = 0; n < 4; ++n) {
      const int rb = tx + 16 * n;
      if (rb < k) out[rb] = acc[m][n];
    }
  }
}

// ------------------------------------------------------------------------------ tensor-core form (bf16 tables)
// The same product on the fifth-generation tensor cores, exact enough for the 1e-5 bar because no operand is
// rounded: psi is bf16 as stored, and every scaled entry x = fl32(g[r] * phi[a][r]) (a 24-bit significand) is cut
// into three bf16 pieces, x = hi + mid + lo exactly (each piece is the round-to-nearest bf16 of what is left), so
// the three products with psi are exact and only the fp32 accumulation in tensor memory rounds.
//
// One CTA of 256 threads per (sequence, position), R <= 256 in one pass or in passes of 128: the warps gather the k predecessor
// rows of phi and the k successor rows of psi (eight rows in flight per warp), scale and split phi and store the
// operands as K-major tiles of 128-byte rows under the 128-byte swizzle -- A1 = [hi; mid] and A2 = [lo; 0] of 128
// rows each, B = psi of 64 rows, one 64-element slab of K after the other (82 KB: two CTAs per SM, so one CTA's
// gather hides behind the other's product).  One thread issues 2 x R / 16 tcgen05.mma (M = 128, N = 64, K = 16)
// into 64 columns of tensor memory: rows 0-63 of the accumulator collect (hi + lo) psi^T and rows 64-127
// mid psi^T; the epilogue reads both with tcgen05.ld, adds them through shared memory and writes the k x k block
// with coalesced stores.  The waits for the MMAs are bounded.
constexpr int ST_T = 256;
constexpr int ST_SPIN = 1 << 22;
constexpr int ST_A_SLAB = 128 * 128, ST_B_SLAB = 64 * 128;  // bytes of one K slab of an operand
constexpr int ST_EX_LD = 65;                                 // floats per row of the epilogue's exchange buffer
constexpr int ST_SP = 2;                                     // K slabs (of 64) per pass

static __device__ unsigned int g_sel_timeouts;

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__global__ void __launch_bounds__(ST_T, 2)
k_selector_scores_tc(const __nv_bfloat16* __restrict__ phi, const __nv_bfloat16* __restrict__ psi, int V, int R,
                     const float* __restrict__ gate, const int32_t* __restrict__ cand_ids,
                     const int32_t* __restrict__ anchor_tokens, int L, int k, float* __restrict__ bigram,
                     float* __restrict__ anchor_bigram, int slabs_per_pass) {
  extern __shared__ unsigned char sel_raw[];
  __shared__ int s_pred[GS_K], s_succ[GS_K];
  __shared__ uint64_t s_bar;
  __shared__ uint32_t s_tmem;
  const int b = blockIdx.x / L, i = blockIdx.x % L;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (i == 0 && (anchor_tokens == nullptr || anchor_bigram == nullptr)) return;  // (the whole CTA)
  unsigned char* base = sel_raw + ((1024u - (tc_smem(sel_raw) & 1023u)) & 1023u);  // tiles start on 1024 bytes
  const int nslab = R / 64, sp = slabs_per_pass, npass = (nslab + sp - 1) / sp;
  unsigned char* A1 = base;
  unsigned char* A2 = A1 + sp * ST_A_SLAB;
  unsigned char* Bt = A2 + sp * ST_A_SLAB;
  const int npred = i == 0 ? 1 : k;
  if (tid < GS_K) {
    int a = -1, t = -1;
    if (tid < npred) a = i == 0 ? anchor_tokens[b] : cand_ids[((int64_t)b * L + i - 1) * k + tid];
    if (tid < k) t = cand_ids[((int64_t)b * L + i) * k + tid];
    // memory-safe for ids outside the vocabulary; -1 marks a row that does not exist
    s_pred[tid] = tid < npred ? (a < 0 ? 0 : (a >= V ? V - 1 : a)) : -1;
    s_succ[tid] = tid < k ? (t < 0 ? 0 : (t >= V ? V - 1 : t)) : -1;
  }
  if (tid == 0) {
    tc_bar_init(&s_bar, 1);
    tc_bar_init_fence();
  }
  if (warp == 0) tc_tmem_alloc(&s_tmem, 64u);
  // rows 64-127 of A2 stay zero
  for (int q = tid; q < sp * 64 * 8; q += ST_T) {
    const int sl = q / 512, row = 64 + (q % 512) / 8, c = q % 8;
    *reinterpret_cast<uint4*>(A2 + sl * ST_A_SLAB + tc_swizzled(row, c)) = make_uint4(0u, 0u, 0u, 0u);
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = s_tmem;

  // this lane's eight elements of a table row: r = 8 lane ... 8 lane + 7, i.e. chunk lane % 8 of slab lane / 8
  const bool have = lane * 8 < R;
  const int sl = lane >> 3, ch = lane & 7;
  float g[8];
  {
    const float* gp = gate + ((int64_t)b * L + i) * R + lane * 8;
    const float4 g0 = have ? *reinterpret_cast<const float4*>(gp) : make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 g1 = have ? *reinterpret_cast<const float4*>(gp + 4) : make_float4(0.f, 0.f, 0.f, 0.f);
    g[0] = g0.x; g[1] = g0.y; g[2] = g0.z; g[3] = g0.w; g[4] = g1.x; g[5] = g1.y; g[6] = g1.z; g[7] = g1.w;
  }
  uint32_t acc = 0u;  // (thread 0: the first product of the first pass overwrites the accumulator)
  for (int pk = 0; pk < npass; ++pk) {
    const bool mine = have && (sl / sp) == pk;  // this lane's elements belong to this pass
    const int ls = sl % sp;                      // ... and to this slab of the pass
#pragma unroll
    for (int half = 0; half < 2; ++half) {  // the phi operand, then the psi operand; a warp takes eight rows of each
      uint4 raw[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int row = warp * 8 + q;
        const int tok = half == 0 ? s_pred[row] : s_succ[row];
        const __nv_bfloat16* src = (half == 0 ? phi : psi) + (int64_t)(tok < 0 ? 0 : tok) * R + lane * 8;
        raw[q] = (tok >= 0 && mine) ? __ldg(reinterpret_cast<const uint4*>(src)) : make_uint4(0u, 0u, 0u, 0u);
      }
      if (!mine) continue;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int row = warp * 8 + q;
        if (half == 1) {
          *reinterpret_cast<uint4*>(Bt + ls * ST_B_SLAB + tc_swizzled(row, ch)) = raw[q];
          continue;
        }
        Frag<__nv_bfloat16> fr;
        fr.unpack(raw[q]);
        float hi[8], mid[8], lo[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float x = __fmul_rn(g[j], fr.x[j]);
          hi[j] = __bfloat162float(__float2bfloat16_rn(x));
          const float r1 = __fsub_rn(x, hi[j]);   // exact
          mid[j] = __bfloat162float(__float2bfloat16_rn(r1));
          lo[j] = __fsub_rn(r1, mid[j]);          // exact, and a bf16 value itself
        }
        const uint4 vh = make_uint4(pack_bf16x2(hi[0], hi[1]), pack_bf16x2(hi[2], hi[3]), pack_bf16x2(hi[4], hi[5]), pack_bf16x2(hi[6], hi[7]));
        const uint4 vm = make_uint4(pack_bf16x2(mid[0], mid[1]), pack_bf16x2(mid[2], mid[3]), pack_bf16x2(mid[4], mid[5]), pack_bf16x2(mid[6], mid[7]));
        const uint4 vl = make_uint4(pack_bf16x2(lo[0], lo[1]), pack_bf16x2(lo[2], lo[3]), pack_bf16x2(lo[4], lo[5]), pack_bf16x2(lo[6], lo[7]));
        *reinterpret_cast<uint4*>(A1 + ls * ST_A_SLAB + tc_swizzled(row, ch)) = vh;
        *reinterpret_cast<uint4*>(A1 + ls * ST_A_SLAB + tc_swizzled(row + 64, ch)) = vm;
        *reinterpret_cast<uint4*>(A2 + ls * ST_A_SLAB + tc_swizzled(row, ch)) = vl;
      }
    }
    tc_fence_smem_to_async();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after_sync();
      constexpr uint32_t idesc = tc_idesc_bf16(128, 64);
      const uint32_t a1 = tc_smem(A1), a2 = tc_smem(A2), bt = tc_smem(Bt);
      const int ns = nslab - pk * sp < sp ? nslab - pk * sp : sp;  // slabs of this pass
      for (int pass = 0; pass < 2; ++pass)
        for (int s2 = 0; s2 < ns; ++s2)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {  // 16 bf16 = 32 bytes along K inside the swizzled row
            tc_mma(tmem, tc_desc((pass == 0 ? a1 : a2) + s2 * ST_A_SLAB + kk * 32), tc_desc(bt + s2 * ST_B_SLAB + kk * 32), idesc, acc);
            acc = 1u;
          }
      tc_commit(&s_bar);
    }
    // the operand tiles may be overwritten (next pass, epilogue) once these products are done
    const bool done = tc_bar_wait(&s_bar, (uint32_t)pk & 1u, ST_SPIN);
    if (!done && tid == 0) atomicAdd(&g_sel_timeouts, 1u);
    tc_fence_after_sync();
  }
  // ---- epilogue: accumulator rows 0-63 and 64-127 are added through shared memory (the operand tiles are free now)
  float* ex = reinterpret_cast<float*>(base);
  uint32_t v0[32], v1[32];
  if (warp < 4) {
    const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16);
    tc_tmem_ld32(taddr, v0);
    tc_tmem_ld32(taddr + 32u, v1);
    if (warp >= 2) {
      float* dst = ex + ((warp - 2) * 32 + lane) * ST_EX_LD;
#pragma unroll
      for (int c = 0; c < 32; ++c) { dst[c] = __uint_as_float(v0[c]); dst[32 + c] = __uint_as_float(v1[c]); }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp < 2) {
    float* dst = ex + (warp * 32 + lane) * ST_EX_LD;
#pragma unroll
    for (int c = 0; c < 32; ++c) { dst[c] += __uint_as_float(v0[c]); dst[32 + c] += __uint_as_float(v1[c]); }
  }
  __syncthreads();
  float* out = i == 0 ? anchor_bigram + (int64_t)b * k : bigram + ((int64_t)b * (L - 1) + i - 1) * k * k;
  for (int e = tid; e < npred * k; e += ST_T) {
    const int ra = e / k, rb = e - ra * k;
    out[e] = ex[ra * ST_EX_LD + rb];
  }
  if (warp == 0) {
    tc_fence_after_sync();
    tc_tmem_dealloc(tmem, 64u);
  }
}

cudaError_t selector_timeouts(unsigned int* out) { return cudaMemcpyFromSymbol(out, g_sel_timeouts, sizeof *out); }

cudaError_t launch_selector_scores(const void* phi, const void* psi, int dtype, int V, int R, const float* gate,
                                   const int32_t* cand_ids, const int32_t* anchor_tokens, int B, int L, int k,
                                   float* bigram, float* anchor_bigram, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const size_t smem = (size_t)2 * GS_K * GS_LD * sizeof(float);
  if (dtype == UBT_BF16 && R % 64 == 0 && R <= 256 && k <= GS_K) {
    // few CTAs: the whole of K in one pass (shortest CTA); many: passes of 128, so that two CTAs share an SM and
    // one's gather hides behind the other's product
    const int nslab = R / 64;
    const int sp = (B * L <= device_info().sm_count || nslab < ST_SP) ? nslab : ST_SP;
    const size_t smem_tc = (size_t)sp * (2 * ST_A_SLAB + ST_B_SLAB) + 1024;
    cudaError_t e = allow_max_dynamic_smem<k_selector_scores_tc>();
    if (e != cudaSuccess) return e;
    k_selector_scores_tc<<<B * L, ST_T, smem_tc, st>>>(static_cast<const __nv_bfloat16*>(phi),
                                                      static_cast<const __nv_bfloat16*>(psi), V, R, gate, cand_ids,
                                                      anchor_tokens, L, k, bigram, anchor_bigram, sp);
    return cudaGetLastError();
  }
  if (dtype == UBT_BF16) {
    auto kern = k_selector_scores<__nv_bfloat16>;
    cudaError_t e = allow_max_dynamic_smem<k_selector_scores<__nv_bfloat16>>();
    if (e != cudaSuccess) return e;
    kern<<<B * L, GS_T, smem, st>>>(static_cast<const __nv_bfloat16*>(phi), static_cast<const __nv_bfloat16*>(psi), V,
                                    R, gate, cand_ids, anchor_tokens, L, k, bigram, anchor_bigram);
  } else {
    auto kern = k_selector_scores<float>;
    cudaError_t e = allow_max_dynamic_smem<k_selector_scores<float>>();
    if (e != cudaSuccess) return e;
    kern<<<B * L, GS_T, smem, st>>>(static_cast<const float*>(phi), static_cast<const float*>(psi), V, R, gate,
                                    cand_ids, anchor_tokens, L, k, bigram, anchor_bigram);
  }
  return cudaGetLastError();
}

}  // namespace ubt
