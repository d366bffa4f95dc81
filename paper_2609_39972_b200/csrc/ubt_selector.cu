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
#include "ubt_internal.h"

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

cudaError_t launch_selector_scores(const void* phi, const void* psi, int dtype, int V, int R, const float* gate,
                                   const int32_t* cand_ids, const int32_t* anchor_tokens, int B, int L, int k,
                                   float* bigram, float* anchor_bigram, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const size_t smem = (size_t)2 * GS_K * GS_LD * sizeof(float);
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
