// Step a4, path-only form (Appendix A, verification): the walk needs the target's pick only at the slots it
// visits -- the root, then one accepted child after the other -- so this kernel evaluates at most L + 1 of the N
// target rows of a sequence instead of all of them.  Same verdict as the all-rows form, a fraction of the bytes.
//
// The picks depend on one another (the next row is known only once the current pick is), so the walk is a chain
// of steps.  One cooperative launch runs the whole chain: every CTA keeps the walk state of every sequence (it is
// a pure function of the picks, so all CTAs agree without exchanging it), every step cuts the current rows of
// the sequences still walking into one slice per CTA, the slices' results meet in global memory, and a grid-wide
// barrier separates the steps.  Greedy: one barrier per step (the slice maxima meet through a 64-bit atomic
// maximum).  Sampling: three (row maximum; integer weight sums per slice; the slice that holds the Philox
// threshold finds the token), with the arithmetic of the all-rows kernels, so the picks are bit-identical.
//
// The grid barrier is a counter in the caller's workspace (zeroed by a memset node in front of the kernel) that
// only grows; a CTA waits for it with a bounded number of polls and gives up by raising the status bit of every
// sequence, so a lost CTA cannot hang the others.
#include "ubt_internal.h"
#include "ubt_pick.cuh"

namespace ubt {

constexpr int VP_T = 256;            // threads per CTA
constexpr int kPathMaxB = 1024;      // sequences whose walk state fits in a CTA's shared memory
constexpr int kPathSpinLimit = 1 << 18;

static __device__ unsigned int g_path_timeouts;  // bounded grid-barrier waits that gave up (0 in a healthy run)

struct PathWs {
  unsigned int* counter;            // [1] grid barrier
  unsigned long long* key;          // greedy: [B, steps] slice maxima met by atomicMax
  uint32_t* rowmax;                 // sampling: [B, steps] ordering key of the row maximum
  unsigned long long* psum;         // sampling: [B, grid] integer weight sum of every slice
  int32_t* pick;                    // sampling: [B, steps]
  int steps;                        // L + 1
};

// All threads of the grid call this; returns false if the wait gave up (every thread of the CTA agrees).
__device__ __forceinline__ bool grid_barrier(unsigned int* counter, unsigned int target, int* s_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(counter, 1u);
    bool ok = false;
    for (int spins = 0; spins < kPathSpinLimit; ++spins) {
      unsigned int seen;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
      if (seen >= target) { ok = true; break; }
      __nanosleep(64);
    }
    if (!ok) { atomicAdd(&g_path_timeouts, 1u); *s_flag = 1; }
  }
  __syncthreads();
  return *reinterpret_cast<volatile int*>(s_flag) == 0;
}

// Columns [c0, c1) of a row that CTA `cta` of `grid` handles: whole fragments of VEC elements, the ragged rest of
// the row goes to the last CTA.
__device__ __forceinline__ void slice_of(int V, int vec, int cta, int grid, int& c0, int& c1) {
  const int frags = V / vec;
  const int per = (frags + grid - 1) / grid;
  const int f0 = min(cta * per, frags), f1 = min(f0 + per, frags);
  c0 = f0 * vec;
  c1 = cta == grid - 1 ? V : f1 * vec;
}

template <typename T, int MODE>
__global__ void __launch_bounds__(VP_T, 1)
k_verify_path(ubt_tree tree, const T* __restrict__ logits, int V, uint64_t seed, float temperature, PathWs w,
              ubt_verify_result out, int32_t* __restrict__ node_pick, int32_t* __restrict__ status) {
  __shared__ unsigned char s_cur[kPathMaxB], s_acc[kPathMaxB], s_live[kPathMaxB];
  __shared__ int s_flag, s_nlive;
  constexpr int VEC = 16 / (int)sizeof(T);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NW = VP_T / 32;
  const int B = tree.B, N = tree.N, L = tree.L, G = gridDim.x, cta = blockIdx.x;
  const bool vec_ok = V % VEC == 0;
  int c0, c1;
  slice_of(V, vec_ok ? VEC : 1, cta, G, c0, c1);
  for (int b = tid; b < B; b += VP_T) { s_cur[b] = 0; s_acc[b] = 0; s_live[b] = 1; }
  if (tid == 0) s_flag = 0;
  __syncthreads();
  if (cta == 0) {  // outputs start as "nothing accepted"; the walk fills them in
    for (int i = tid; i < B * (L + 1); i += VP_T) {
      out.accepted_nodes[i] = i % (L + 1) == 0 ? 0 : -1;
      out.out_tokens[i] = -1;
    }
    if (node_pick)
      for (int i = tid; i < B * N; i += VP_T) node_pick[i] = -1;
    if (status)
      for (int b = tid; b < B; b += VP_T) status[b] = 0;
  }
  unsigned int phase = 0;
  const float inv_t = __fdiv_rn(1.0f, temperature);
  const float a = __fmul_rn(0x1.715476p+0f, inv_t);

  // maximum (value, lowest column) of this CTA's slice of row `rowp`, as an ordering key; all lanes get it
  auto slice_max_key = [&](const T* rowp) -> unsigned long long {
    float best = -INFINITY;
    int bcol = -1;
    bool saw_nan = false;
    if (vec_ok) {
      const uint4* frag = reinterpret_cast<const uint4*>(rowp);
      for (int f = c0 / VEC + lane; f < c1 / VEC; f += 32) {
        const uint4 v = ldg_stream(frag + f);
        const float fm = frag_max(v, (const T*)nullptr);
        saw_nan = saw_nan || fm != fm;
        if (fm > best) {  // columns ascend within a lane: strict > keeps the lowest column
          Frag<T> x;
          x.unpack(v);
          int j0 = 0;
#pragma unroll
          for (int j = VEC - 1; j >= 0; --j) j0 = x.x[j] == fm ? j : j0;
          best = fm;
          bcol = f * VEC + j0;
        }
      }
    } else {
      for (int c = c0 + lane; c < c1; c += 32) {
        const float x = load_elem(rowp, c);
        saw_nan = saw_nan || x != x;
        if (x > best) { best = x; bcol = c; }
      }
    }
    unsigned long long key = bcol >= 0 ? make_key(best, bcol) : 0ull;
    key = saw_nan ? kKeyNaNSeen : key;
    return warp_max_u64(key);
  };

  for (int step = 0; step <= L; ++step) {
    // ---- phase 1: every sequence still walking, one warp at a time: this CTA's slice of its current row
    for (int b = warp; b < B; b += NW) {
      if (!s_live[b]) continue;
      const T* rowp = logits + ((int64_t)b * N + s_cur[b]) * V;
      const unsigned long long key = slice_max_key(rowp);
      if (lane == 0 && key != 0ull) {
        if (MODE == UBT_VERIFY_GREEDY) atomicMax(&w.key[(int64_t)b * w.steps + step], key);
        else atomicMax(&w.rowmax[(int64_t)b * w.steps + step], (uint32_t)(key >> 32));
      }
    }
    if (!grid_barrier(w.counter, ++phase * G, &s_flag)) break;

    if (MODE == UBT_VERIFY_SAMPLE) {
      // ---- phase 2: integer weight sum of this CTA's slice (the weights of the all-rows kernels)
      for (int b = warp; b < B; b += NW) {
        if (!s_live[b]) continue;
        const uint32_t mk = __ldcg(&w.rowmax[(int64_t)b * w.steps + step]);
        const float m = key2f(mk);
        unsigned long long acc = 0;
        if (mk != 0u && mk < 0xff800000u) {  // a finite maximum (else: reported below, weights unused)
          const float c = -__fmul_rn(m, a);
          const T* rowp = logits + ((int64_t)b * N + s_cur[b]) * V;
          for (int col = c0 + lane; col < c1; col += 32) acc += weight_of(load_elem(rowp, col), a, c);
          acc = warp_sum_u64(acc);
        }
        if (lane == 0) w.psum[(int64_t)b * G + cta] = acc;
      }
      if (!grid_barrier(w.counter, ++phase * G, &s_flag)) break;
      // ---- phase 3: the slice that holds the row's Philox threshold finds the token
      for (int b = warp; b < B; b += NW) {
        if (!s_live[b]) continue;
        const uint32_t mk = __ldcg(&w.rowmax[(int64_t)b * w.steps + step]);
        if (mk == 0u || mk >= 0xff800000u) {  // NaN or +inf in the row (or nothing comparable): no pick
          if (cta == 0 && lane == 0) w.pick[(int64_t)b * w.steps + step] = -1;
          continue;
        }
        // totals and the prefix in front of this CTA's slice
        unsigned long long before = 0, total = 0;
        for (int g = lane; g < G; g += 32) {
          const unsigned long long v = __ldcg(&w.psum[(int64_t)b * G + g]);
          total += v;
          before += g < cta ? v : 0ull;
        }
        total = warp_sum_u64(total);
        before = warp_sum_u64(before);
        const unsigned long long mine = __ldcg(&w.psum[(int64_t)b * G + cta]);
        uint32_t x[4];
        philox4x32_10((uint32_t)s_cur[b], (uint32_t)b, 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
        const unsigned long long R = (unsigned long long)x[0] | ((unsigned long long)x[1] << 32);
        const unsigned long long theta = __umul64hi(R, total);
        if (!(theta >= before && theta < before + mine)) continue;  // another slice holds it
        const float m = key2f(mk);
        const float c = -__fmul_rn(m, a);
        const T* rowp = logits + ((int64_t)b * N + s_cur[b]) * V;
        // consecutive runs of columns per lane, then a scan over the lanes, then the token inside one run
        const int len = c1 - c0, per = (len + 31) / 32;
        const int t0 = c0 + lane * per, t1 = min(t0 + per, c1);
        unsigned long long lsum = 0;
        for (int col = t0; col < t1; ++col) lsum += weight_of(load_elem(rowp, col), a, c);
        unsigned long long inc = lsum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned long long up = __shfl_up_sync(FULL, inc, o);
          if (lane >= o) inc += up;
        }
        const unsigned long long rel = theta - before;
        const unsigned hit = __ballot_sync(FULL, inc > rel);
        const int l = hit ? __ffs(hit) - 1 : 31;
        if (lane == l) {
          unsigned long long run = inc - lsum;
          int ans = t1 - 1;
          for (int col = t0; col < t1; ++col) {
            run += weight_of(load_elem(rowp, col), a, c);
            if (run > rel) { ans = col; break; }
          }
          ans = ans < 0 ? 0 : (ans >= V ? V - 1 : ans);
          w.pick[(int64_t)b * w.steps + step] = ans;
        }
      }
      if (!grid_barrier(w.counter, ++phase * G, &s_flag)) break;
    }

    // ---- every CTA advances every walk by the step's pick (identical in all CTAs)
    if (tid == 0) s_nlive = 0;
    __syncthreads();
    for (int b = warp; b < B; b += NW) {
      if (!s_live[b]) continue;
      int x, bits = 0;
      if (MODE == UBT_VERIFY_GREEDY) {
        const unsigned long long key = __ldcg(&w.key[(int64_t)b * w.steps + step]);
        x = key ? key_idx(key) : 0;
        if (key >= kKeyPlusInf) bits = kStatusNonFinite;
      } else {
        x = __ldcg(&w.pick[(int64_t)b * w.steps + step]);
        if (x < 0) { bits = kStatusNonFinite; x = 0; }
      }
      const int cur = s_cur[b], acc = s_acc[b], n_nodes = tree.n_nodes[b];
      const int64_t o = (int64_t)b * N;
      int child = -1;
      for (int cc = 1; cc < n_nodes && child < 0; cc += 32) {
        const int c = cc + lane;
        const bool match = c < n_nodes && tree.parents[o + c] == cur && tree.token_ids[o + c] == x;
        const unsigned mm = __ballot_sync(FULL, match);
        if (mm) child = cc + __ffs(mm) - 1;
      }
      const bool stop = child < 0 || acc == L;
      if (lane == 0) {
        if (cta == 0) {
          out.out_tokens[(int64_t)b * (L + 1) + acc] = x;
          if (node_pick) node_pick[o + cur] = x;
          if (bits && status) atomicOr(&status[b], bits);
          if (stop) { out.bonus_token[b] = x; out.accepted_len[b] = acc; }
          else out.accepted_nodes[(int64_t)b * (L + 1) + acc + 1] = child;
        }
        if (stop) s_live[b] = 0;
        else { s_cur[b] = (unsigned char)child; s_acc[b] = (unsigned char)(acc + 1); atomicAdd(&s_nlive, 1); }
      }
    }
    __syncthreads();
    if (s_nlive == 0) break;
  }
  if (*reinterpret_cast<volatile int*>(&s_flag) && cta == 0 && status) {  // a barrier wait gave up
    __syncthreads();
    for (int b = tid; b < B; b += VP_T) atomicOr(&status[b], kStatusWaitGaveUp);
  }
}

// ------------------------------------------------------------------------------------ host side
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static int path_steps(int N) { return (N < kMaxL + 1 ? N : kMaxL + 1); }  // a walk visits at most min(N, L + 1) slots

size_t verify_path_workspace_bytes(int B, int N, int mode) {
  const size_t steps = (size_t)path_steps(N), grid = (size_t)device_info().sm_count;
  size_t bytes = 256;  // the barrier counter
  if (mode == UBT_VERIFY_GREEDY) return bytes + align_up((size_t)B * steps * 8, 256);
  return bytes + align_up((size_t)B * steps * 4, 256) + align_up((size_t)B * grid * 8, 256) +
         align_up((size_t)B * steps * 4, 256);
}

template <typename T, int MODE>
static cudaError_t launch_verify_path_t(const ubt_tree& tree, const void* logits, int V, uint64_t seed, float temperature,
                                        void* ws, int32_t* node_pick, const ubt_verify_result& out, int32_t* status,
                                        cudaStream_t st) {
  const int B = tree.B, steps = path_steps(tree.N), grid = device_info().sm_count;
  unsigned char* p = static_cast<unsigned char*>(ws);
  PathWs w{};
  w.steps = steps;
  w.counter = reinterpret_cast<unsigned int*>(p); p += 256;
  size_t zero_bytes = 256;
  if (MODE == UBT_VERIFY_GREEDY) {
    w.key = reinterpret_cast<unsigned long long*>(p);
    zero_bytes += align_up((size_t)B * steps * 8, 256);
  } else {
    w.rowmax = reinterpret_cast<uint32_t*>(p); p += align_up((size_t)B * steps * 4, 256);
    zero_bytes += align_up((size_t)B * steps * 4, 256);
    w.psum = reinterpret_cast<unsigned long long*>(p); p += align_up((size_t)B * grid * 8, 256);
    w.pick = reinterpret_cast<int32_t*>(p);
  }
  // the counter and the atomic-maximum slots start at zero (a memset node on the stream, no allocation)
  cudaError_t e = cudaMemsetAsync(ws, 0, zero_bytes, st);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(VP_T);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident together: the grid barrier needs it
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_verify_path<T, MODE>, tree, static_cast<const T*>(logits), V, seed, temperature, w,
                            out, node_pick, status);
}

cudaError_t launch_verify_path(const ubt_tree& tree, const void* logits, int dtype, int V, int mode, uint64_t seed,
                               float temperature, void* ws, int32_t* node_pick, const ubt_verify_result& out,
                               int32_t* status, cudaStream_t st) {
  if (tree.B == 0) return cudaSuccess;
  if (dtype == UBT_BF16) {
    return mode == UBT_VERIFY_GREEDY
               ? launch_verify_path_t<__nv_bfloat16, UBT_VERIFY_GREEDY>(tree, logits, V, seed, temperature, ws, node_pick, out, status, st)
               : launch_verify_path_t<__nv_bfloat16, UBT_VERIFY_SAMPLE>(tree, logits, V, seed, temperature, ws, node_pick, out, status, st);
  }
  return mode == UBT_VERIFY_GREEDY
             ? launch_verify_path_t<float, UBT_VERIFY_GREEDY>(tree, logits, V, seed, temperature, ws, node_pick, out, status, st)
             : launch_verify_path_t<float, UBT_VERIFY_SAMPLE>(tree, logits, V, seed, temperature, ws, node_pick, out, status, st);
}

int verify_path_max_batch() { return kPathMaxB; }

cudaError_t ring_timeouts_path(unsigned int* out) { return cudaMemcpyFromSymbol(out, g_path_timeouts, sizeof *out); }

}  // namespace ubt
