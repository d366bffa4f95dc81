// Step a4: the target's pick at every tree slot, then the acceptance walk (Appendix A, verification).
//
// Greedy: B*N*V target logits are cut into equal contiguous spans, one per CTA; each CTA emits, for
// every row segment it meets, the (value, lowest token) maximum as one 64-bit key.  The walk kernel
// reduces a row's few keys, so no atomics and no zero-initialised scratch are needed.
// Sampling: one CTA per row; pass 1 finds the row maximum, pass 2 (served from L2) turns every logit
// into an integer weight with a fixed sequence of IEEE operations and sums them per 1024-token chunk;
// the chunk holding the Philox threshold is rescanned to find the token.  Integer sums make the pick
// independent of the order of addition.
#include "ubt_internal.h"

namespace ubt {

constexpr int G4_T = 512;
constexpr int G4_U = 4;

template <typename T, int VEC>
__device__ __forceinline__ void load_row_frag(const T* seg, int nfrag, int i, uint4& raw, float& sc) {
  if constexpr (VEC == 1) {
    sc = i < nfrag ? load_elem(seg, i) : -INFINITY;
  } else {
    if (i < nfrag) {
      raw = ldg_stream(reinterpret_cast<const uint4*>(seg) + i);
    } else {
      const uint32_t ninf = sizeof(T) == 2 ? 0xff80ff80u : 0xff800000u;
      raw = make_uint4(ninf, ninf, ninf, ninf);
    }
  }
}

template <typename T, int VEC>
__device__ __forceinline__ void frag_values(const uint4& raw, float sc, float (&x)[VEC]) {
  if constexpr (VEC == 1) {
    x[0] = sc;
  } else {
    Frag<T> f;
    f.unpack(raw);
#pragma unroll
    for (int j = 0; j < VEC; ++j) x[j] = f.x[j];
  }
}

// ---------------------------------------------------------------------------- greedy picks
template <typename T, int VEC>
__global__ void __launch_bounds__(G4_T, VEC == 1 ? 1 : 2)
k_row_argmax(const T* __restrict__ logits, int64_t total, int V, SpanPlan plan,
             unsigned long long* __restrict__ part_key) {
  __shared__ unsigned long long red[G4_T / 32];
  constexpr int TILE_FRAGS = G4_T * G4_U;
  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t lo = (int64_t)blockIdx.x * plan.span;
  const int64_t hi = lo + plan.span < total ? lo + plan.span : total;

  for (int64_t e = lo; e < hi;) {
    const int64_t row = e / V;
    const int c0 = (int)(e - row * V);
    const int c1 = (int)((int64_t)V - c0 < hi - e ? V : c0 + (hi - e));
    const T* seg = logits + row * V + c0;
    const int nfrag = (c1 - c0) / VEC;
    e += c1 - c0;

    // Baseline (-inf, the thread's first column): true if all its elements are -inf, replaced otherwise.
    float best = -INFINITY;
    int bcol = c0 + tid * VEC;
    const bool has = tid < nfrag;
    uint4 cur[G4_U], nxt[G4_U];
    float curs[G4_U], nxts[G4_U];
#pragma unroll
    for (int u = 0; u < G4_U; ++u) load_row_frag<T, VEC>(seg, nfrag, u * G4_T + tid, cur[u], curs[u]);
    for (int base = 0; base < nfrag; base += TILE_FRAGS) {
      if (base + TILE_FRAGS < nfrag) {
#pragma unroll
        for (int u = 0; u < G4_U; ++u)
          load_row_frag<T, VEC>(seg, nfrag, base + TILE_FRAGS + u * G4_T + tid, nxt[u], nxts[u]);
      }
#pragma unroll
      for (int u = 0; u < G4_U; ++u) {
        float x[VEC];
        frag_values<T, VEC>(cur[u], curs[u], x);
        float vmax = x[0];
#pragma unroll
        for (int j = 1; j < VEC; ++j) vmax = fmaxf(vmax, x[j]);
        if (vmax > best) {  // columns ascend within a thread: strict > keeps the lowest token
          const int col0 = c0 + (base + u * G4_T + tid) * VEC;
#pragma unroll
          for (int j = 0; j < VEC; ++j)
            if (x[j] > best) { best = x[j]; bcol = col0 + j; }
        }
      }
#pragma unroll
      for (int u = 0; u < G4_U; ++u) { cur[u] = nxt[u]; curs[u] = nxts[u]; }
    }
    unsigned long long key = has ? make_key(best, bcol) : 0ull;
    key = warp_max_u64(key);
    __syncthreads();
    if (lane == 0) red[tid >> 5] = key;
    __syncthreads();
    if (tid == 0) {
      unsigned long long r = red[0];
      for (int w = 1; w < G4_T / 32; ++w) r = red[w] > r ? red[w] : r;
      const int64_t c_first = (row * (int64_t)V) / plan.span;
      part_key[row * plan.smax + ((int64_t)blockIdx.x - c_first)] = r;
    }
  }
}

// ---------------------------------------------------------------------------- sampling picks
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
    c0 = n0; c1 = l1; c2 = n2; c3 = l0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Integer weight of one logit: trunc(2^(40 + y)), y = max(fma(z, a, c), -42), with 2^y evaluated as
// 2^n * p(f), n = rint(y), f = y - n, p a fixed degree-5 polynomial in fma Horner form.  Every step
// is one IEEE-754 operation, so any machine reproduces the same integer.
__device__ __forceinline__ unsigned long long weight_of(float z, float a, float c) {
  float y = __fmaf_rn(z, a, c);
  y = fmaxf(y, -42.0f);
  const float big = 12582912.0f;
  const float tmp = __fadd_rn(y, big);
  const float nf = __fsub_rn(tmp, big);
  const float f = __fsub_rn(y, nf);
  float p = 0x1.5c7746p-10f;
  p = __fmaf_rn(p, f, 0x1.3cea8p-7f);
  p = __fmaf_rn(p, f, 0x1.c6b54ap-5f);
  p = __fmaf_rn(p, f, 0x1.ebf9bcp-3f);
  p = __fmaf_rn(p, f, 0x1.62e42cp-1f);
  p = __fmaf_rn(p, f, 1.0f);
  // p * 2^(n+40): add (n+40) to the exponent field; tmp's low mantissa bits hold n in two's complement
  const uint32_t e = __float_as_uint(p) + ((__float_as_uint(tmp) + 40u) << 23);
  return __float2ull_rz(__uint_as_float(e));
}

constexpr int G5_T = 512;
constexpr int G5_CHUNK = 1024;     // tokens per partial sum
constexpr int G5_MAXCHUNKS = 2048;  // V <= 2M

template <typename T, int VEC>
__global__ void __launch_bounds__(G5_T, 2)
k_row_sample(const T* __restrict__ logits, int64_t rows, int N, int V, uint64_t seed, float temperature,
             int32_t* __restrict__ pick) {
  __shared__ unsigned long long csum[G5_MAXCHUNKS];
  __shared__ float redf[G5_T / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nchunks = (V + G5_CHUNK - 1) / G5_CHUNK;
  constexpr int CF = G5_CHUNK / VEC;  // fragments per chunk

  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    const T* rowp = logits + row * V;
    const int nfrag = V / VEC;  // V % VEC == 0 on the vector path; VEC == 1 otherwise
    // pass 1: row maximum
    float m = -INFINITY;
#pragma unroll 4
    for (int f = tid; f < nfrag; f += G5_T) {
      uint4 raw; float sc = 0.f;
      load_row_frag<T, VEC>(rowp, nfrag, f, raw, sc);
      float x[VEC];
      frag_values<T, VEC>(raw, sc, x);
#pragma unroll
      for (int j = 0; j < VEC; ++j) m = fmaxf(m, x[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(FULL, m, o));
    __syncthreads();
    if (lane == 0) redf[warp] = m;
    __syncthreads();
    m = redf[0];
    for (int w = 1; w < G5_T / 32; ++w) m = fmaxf(m, redf[w]);
    const float inv_t = __fdiv_rn(1.0f, temperature);
    const float a = __fmul_rn(0x1.715476p+0f, inv_t);
    const float c = -__fmul_rn(m, a);

    // pass 2: integer weights, one partial sum per chunk (a warp owns a chunk)
    for (int ch = warp; ch < nchunks; ch += G5_T / 32) {
      unsigned long long acc = 0;
      for (int fi = lane; fi < CF; fi += 32) {
        const int f = ch * CF + fi;
        if (f < nfrag) {
          uint4 raw; float sc = 0.f;
          load_row_frag<T, VEC>(rowp, nfrag, f, raw, sc);
          float x[VEC];
          frag_values<T, VEC>(raw, sc, x);
#pragma unroll
          for (int j = 0; j < VEC; ++j) acc += weight_of(x[j], a, c);
        }
      }
      acc = warp_sum_u64(acc);
      if (lane == 0) csum[ch] = acc;
    }
    __syncthreads();

    // locate the chunk that holds the threshold, then the token inside it (warp 0)
    if (warp == 0) {
      unsigned long long run = 0;
      for (int ch = lane; ch < nchunks; ch += 32) run += csum[ch];
      const unsigned long long total = warp_sum_u64(run);
      uint32_t x[4];
      philox4x32_10((uint32_t)(row % N), (uint32_t)(row / N), 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
      const unsigned long long R = (unsigned long long)x[0] | ((unsigned long long)x[1] << 32);
      unsigned long long theta = __umul64hi(R, total);
      // sequential over groups of 32 chunks, warp scan inside a group
      int found_chunk = nchunks - 1;
      unsigned long long before = 0;
      bool done = false;
      for (int g = 0; g < nchunks && !done; g += 32) {
        const unsigned long long v = (g + lane < nchunks) ? csum[g + lane] : 0ull;
        unsigned long long inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          unsigned long long up = __shfl_up_sync(FULL, inc, o);
          if (lane >= o) inc += up;
        }
        const unsigned hit = __ballot_sync(FULL, before + inc > theta && g + lane < nchunks);
        if (hit) {
          const int l = __ffs(hit) - 1;
          found_chunk = g + l;
          before += __shfl_sync(FULL, inc - v, l);
          done = true;
        } else {
          before += __shfl_sync(FULL, inc, 31);
        }
      }
      theta -= before;  // threshold relative to the chunk start
      // every lane takes 32 consecutive tokens of the chunk
      const int t0 = found_chunk * G5_CHUNK + lane * (G5_CHUNK / 32);
      unsigned long long lsum = 0;
      for (int j = 0; j < G5_CHUNK / 32; ++j) {
        const int tkn = t0 + j;
        lsum += tkn < V ? weight_of(load_elem(rowp, tkn), a, c) : 0ull;
      }
      unsigned long long inc = lsum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned long long up = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += up;
      }
      const unsigned hit = __ballot_sync(FULL, inc > theta);
      const int l = hit ? __ffs(hit) - 1 : 31;
      if (lane == l) {
        unsigned long long run2 = inc - lsum;
        int ans = t0 + G5_CHUNK / 32 - 1;
        for (int j = 0; j < G5_CHUNK / 32; ++j) {
          const int tkn = t0 + j;
          run2 += tkn < V ? weight_of(load_elem(rowp, tkn), a, c) : 0ull;
          if (run2 > theta) { ans = tkn; break; }
        }
        pick[row] = ans < V ? ans : V - 1;
      }
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------- the walk
// One CTA per sequence: gather the picks of its N slots, then warp 0 walks from the root.
__global__ void __launch_bounds__(128)
k_walk(ubt_tree tree, int mode, SpanPlan plan, const unsigned long long* __restrict__ part_key, int V,
       const int32_t* __restrict__ sampled_pick, int32_t* __restrict__ node_pick, ubt_verify_result out) {
  __shared__ int s_pick[kMaxN], s_tok[kMaxN], s_par[kMaxN];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, N = tree.N, L = tree.L;
  const int64_t o = (int64_t)b * N;
  for (int n = tid; n < N; n += blockDim.x) {
    int p;
    if (mode == UBT_VERIFY_GREEDY) {
      const int64_t row = o + n;
      const int64_t c_first = (row * (int64_t)V) / plan.span;
      const int64_t c_last = ((row + 1) * (int64_t)V - 1) / plan.span;
      unsigned long long best = 0;
      for (int64_t j = 0; j <= c_last - c_first; ++j) {
        const unsigned long long key = part_key[row * plan.smax + j];
        best = key > best ? key : best;
      }
      p = key_idx(best);
    } else {
      p = sampled_pick[o + n];
    }
    s_pick[n] = p;
    s_tok[n] = tree.token_ids[o + n];
    s_par[n] = tree.parents[o + n];
    if (node_pick) node_pick[o + n] = p;
  }
  __syncthreads();
  if (tid >= 32) return;
  const int n_nodes = tree.n_nodes[b];
  int32_t* an = out.accepted_nodes + (int64_t)b * (L + 1);
  int32_t* ot = out.out_tokens + (int64_t)b * (L + 1);
  for (int j = lane; j <= L; j += 32) { an[j] = j == 0 ? 0 : -1; ot[j] = -1; }
  __syncwarp();
  int cur = 0, acc = 0;
  for (int step = 0; step <= L; ++step) {  // a path holds at most L draft tokens
    const int x = s_pick[cur];
    int child = -1;
    for (int c0 = 1; c0 < n_nodes && child < 0; c0 += 32) {
      const int c = c0 + lane;
      const bool match = c < n_nodes && s_par[c] == cur && s_tok[c] == x;
      const unsigned m = __ballot_sync(FULL, match);
      if (m) child = c0 + __ffs(m) - 1;
    }
    if (lane == 0) ot[acc] = x;
    if (child < 0 || acc == L) {
      if (lane == 0) { out.bonus_token[b] = x; out.accepted_len[b] = acc; }
      break;
    }
    ++acc;
    if (lane == 0) an[acc] = child;
    cur = child;
  }
}

// ------------------------------------------------------------------------------------ host side
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static SpanPlan argmax_plan(int64_t rows, int V) {
  return make_span_plan(rows, V, device_info().sm_count * 2, 65536);
}

size_t verify_workspace_bytes(int64_t rows, int V, int mode) {
  if (mode == UBT_VERIFY_GREEDY) {
    const SpanPlan p = argmax_plan(rows, V);
    return align_up((size_t)rows * p.smax * sizeof(unsigned long long), 256);
  }
  return align_up((size_t)rows * sizeof(int32_t), 256);
}

VerifyWorkspace carve_verify_workspace(void* ws, int64_t rows, int V, int mode) {
  VerifyWorkspace w{};
  if (mode == UBT_VERIFY_GREEDY) {
    w.plan = argmax_plan(rows, V);
    w.part_key = static_cast<unsigned long long*>(ws);
  } else {
    w.plan = SpanPlan{0, 0, 0};
    w.pick = static_cast<int32_t*>(ws);
  }
  return w;
}

template <typename T, int VEC>
static cudaError_t launch_row_argmax_t(const void* logits, int64_t rows, int V, const VerifyWorkspace& w,
                                       cudaStream_t st) {
  k_row_argmax<T, VEC><<<w.plan.grid, G4_T, 0, st>>>(static_cast<const T*>(logits), rows * (int64_t)V, V,
                                                     w.plan, w.part_key);
  return cudaGetLastError();
}

cudaError_t launch_row_argmax(const void* logits, int dtype, int64_t rows, int V, const VerifyWorkspace& w,
                              cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  if (dtype == UBT_BF16) {
    if (V % 8 == 0) return launch_row_argmax_t<__nv_bfloat16, 8>(logits, rows, V, w, st);
    return launch_row_argmax_t<__nv_bfloat16, 1>(logits, rows, V, w, st);
  }
  if (V % 4 == 0) return launch_row_argmax_t<float, 4>(logits, rows, V, w, st);
  return launch_row_argmax_t<float, 1>(logits, rows, V, w, st);
}

template <typename T, int VEC>
static cudaError_t launch_row_sample_t(const void* logits, int64_t rows, int N, int V, uint64_t seed,
                                       float temperature, int32_t* pick, cudaStream_t st) {
  int grid = device_info().sm_count * 2;
  if ((int64_t)grid > rows) grid = (int)rows;
  k_row_sample<T, VEC><<<grid, G5_T, 0, st>>>(static_cast<const T*>(logits), rows, N, V, seed, temperature,
                                              pick);
  return cudaGetLastError();
}

cudaError_t launch_row_sample(const void* logits, int dtype, int B, int N, int V, uint64_t seed,
                              float temperature, int32_t* pick, cudaStream_t st) {
  const int64_t rows = (int64_t)B * N;
  if (rows == 0) return cudaSuccess;
  if (dtype == UBT_BF16) {
    if (V % 8 == 0) return launch_row_sample_t<__nv_bfloat16, 8>(logits, rows, N, V, seed, temperature, pick, st);
    return launch_row_sample_t<__nv_bfloat16, 1>(logits, rows, N, V, seed, temperature, pick, st);
  }
  if (V % 4 == 0) return launch_row_sample_t<float, 4>(logits, rows, N, V, seed, temperature, pick, st);
  return launch_row_sample_t<float, 1>(logits, rows, N, V, seed, temperature, pick, st);
}

cudaError_t launch_walk(const ubt_tree& tree, int mode, const VerifyWorkspace& w, int V,
                        const int32_t* sampled_pick, int32_t* node_pick, const ubt_verify_result& out,
                        cudaStream_t st) {
  if (tree.B == 0) return cudaSuccess;
  k_walk<<<tree.B, 128, 0, st>>>(tree, mode, w.plan, w.part_key, V, sampled_pick, node_pick, out);
  return cudaGetLastError();
}

#ifdef UBT_BOUNDS_CHECK
// Debug builds only: first out-of-range index seen by the kernels of this file (flag, site, index, limit).
cudaError_t bounds_report_verify(long long out[4]) {
  BoundsReport r;
  cudaError_t e = cudaMemcpyFromSymbol(&r, g_bounds_report, sizeof r);
  out[0] = r.flag; out[1] = r.site; out[2] = r.index; out[3] = r.limit;
  return e;
}
#endif

}  // namespace ubt
