// Step a4, path-only form (Appendix A, verification): the walk needs the target's pick only at the slots it
// visits -- the root, then one accepted child after the other -- so this kernel evaluates at most L + 1 of the N
// target rows of a sequence instead of all of them.  Same verdict as the all-rows form, a fraction of the bytes.
//
// The picks depend on one another (the next row is known only once the current pick is), so the walk is a chain
// of steps, and what counts is the latency of a step.  One thread-block cluster of eight CTAs walks one sequence,
// independently of all other sequences: in every step the current row is cut into 64 contiguous sub-slices (one
// per warp of the cluster), every warp reduces its sub-slice, the 64 results are written into the shared memory
// of all eight CTAs (distributed shared memory) and one cluster barrier later every CTA holds them all, takes the
// same decision and moves to the same child -- the walk state is a pure function of the picks, so it is never
// exchanged.  Greedy: one barrier per step ((value, ~token) keys, maximum).  Sampling: three (row maximum;
// integer weight sums per sub-slice; the sub-slice that holds the Philox threshold finds the token), with the
// arithmetic of the all-rows kernels, so the picks are bit-identical.
//
// Nothing spins: the only waits are cluster barriers, all CTAs of a cluster are resident together by
// construction, and every CTA executes the same sequence of barriers because every decision that controls the
// loop is computed from the same exchanged values.  No workspace is needed.
#include "ubt_internal.h"
#include "ubt_pick.cuh"

namespace ubt {

constexpr int VP_T = 256;            // threads per CTA
constexpr int VP_NW = VP_T / 32;     // warps per CTA
constexpr int VP_CS = 8;             // CTAs per cluster (the portable maximum)
constexpr int VP_PARTS = VP_CS * VP_NW;  // sub-slices of a row

// ---- cluster primitives
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {  // every thread of every CTA of the cluster
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of `p` (a shared-memory location of this CTA) in the shared memory of CTA `rank` of the cluster
__device__ __forceinline__ uint32_t peer_shared(const void* p, uint32_t rank) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p), r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_peer_u64(uint32_t addr, unsigned long long v) {
  asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
__device__ __forceinline__ void st_peer_s32(uint32_t addr, int v) {
  asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint4 ldg_keep(const uint4* p) {  // the weight pass reads the row again: let L1 keep it
  return __ldg(p);
}

struct PathShared {
  int tok[kMaxN], par[kMaxN];
  // what the warps of the cluster exchange; two copies used in turn (a CTA may be one barrier ahead of another)
  unsigned long long xkey[2][VP_PARTS];   // greedy: sub-slice maximum keys; sampling: sub-slice row-maximum keys
  unsigned long long xsum[2][VP_PARTS];   // sampling: integer weight sums of the sub-slices
  int xpick[2];                           // sampling: the token found by the sub-slice that holds the threshold
};

template <typename T, int MODE>
__global__ void __launch_bounds__(VP_T)
k_verify_path(ubt_tree tree, const T* __restrict__ logits, int V, uint64_t seed, float temperature,
              ubt_verify_result out, int32_t* __restrict__ node_pick, int32_t* __restrict__ status) {
  __shared__ PathShared sh;
  constexpr int VEC = 16 / (int)sizeof(T);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = tree.N, L = tree.L;
  const int b = blockIdx.x / VP_CS;
  const uint32_t rank = cluster_rank();
  const int part = (int)rank * VP_NW + warp;  // this warp's sub-slice: parts are in column order
  const bool vec_ok = V % VEC == 0;
  const bool writer = rank == 0 && warp == 0 && lane == 0;
  const int64_t o = (int64_t)b * N;
  // sub-slice [c0, c1): whole fragments when the rows are made of them
  int c0, c1;
  {
    const int unit = vec_ok ? VEC : 1, units = V / unit;
    const int per = (units + VP_PARTS - 1) / VP_PARTS;
    const int u0 = min(part * per, units), u1 = min(u0 + per, units);
    c0 = u0 * unit;
    c1 = u1 * unit;
  }
  const int n_nodes = tree.n_nodes[b];
  for (int n = tid; n < N; n += VP_T) { sh.tok[n] = tree.token_ids[o + n]; sh.par[n] = tree.parents[o + n]; }
  if (rank == 0) {  // outputs start as "nothing accepted"; the walk fills them in
    for (int i = tid; i <= L; i += VP_T) {
      out.accepted_nodes[(int64_t)b * (L + 1) + i] = i == 0 ? 0 : -1;
      out.out_tokens[(int64_t)b * (L + 1) + i] = -1;
    }
    if (node_pick)
      for (int i = tid; i < N; i += VP_T) node_pick[o + i] = -1;
  }
  __syncthreads();
  cluster_sync_all();  // every CTA of the cluster has started: its shared memory may be written from now on

  const float inv_t = __fdiv_rn(1.0f, temperature);
  const float a = __fmul_rn(0x1.715476p+0f, inv_t);
  int cur = 0, acc = 0, bits_all = 0;

  for (int step = 0; step <= L; ++step) {
    const int cp = step & 1;
    const T* rowp = logits + (o + cur) * V;
    // ---- maximum (value, lowest column) of the sub-slice as an ordering key
    unsigned long long key;
    {
      float best = -INFINITY;
      int bcol = -1;
      bool saw_nan = false;
      if (vec_ok) {
        const uint4* frag = reinterpret_cast<const uint4*>(rowp);
        for (int f = c0 / VEC + lane; f < c1 / VEC; f += 32) {
          const uint4 v = MODE == UBT_VERIFY_GREEDY ? ldg_stream(frag + f) : ldg_keep(frag + f);
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
      key = bcol >= 0 ? make_key(best, bcol) : 0ull;
      key = saw_nan ? kKeyNaNSeen : key;
      key = warp_max_u64(key);
    }
    if (lane < VP_CS) st_peer_u64(peer_shared(&sh.xkey[cp][part], (uint32_t)lane), key);
    cluster_sync_all();
    unsigned long long rowkey = sh.xkey[cp][lane] > sh.xkey[cp][lane + 32] ? sh.xkey[cp][lane] : sh.xkey[cp][lane + 32];
    rowkey = warp_max_u64(rowkey);

    int x, bits = 0;
    if (MODE == UBT_VERIFY_GREEDY) {
      x = rowkey ? key_idx(rowkey) : 0;
      if (rowkey >= kKeyPlusInf) bits = kStatusNonFinite;
    } else {
      const uint32_t mk = (uint32_t)(rowkey >> 32);
      if (mk == 0u || mk >= 0xff800000u) {  // NaN or +inf in the row (or nothing comparable): no pick
        x = 0;
        bits = kStatusNonFinite;
      } else {
        // ---- integer weight sum of the sub-slice (the weights of the all-rows kernels)
        const float m = key2f(mk);
        const float c = -__fmul_rn(m, a);
        unsigned long long wsum = 0;
        if (vec_ok) {
          const uint4* frag = reinterpret_cast<const uint4*>(rowp);
          for (int f = c0 / VEC + lane; f < c1 / VEC; f += 32) {
            Frag<T> fr;
            fr.unpack(ldg_keep(frag + f));
#pragma unroll
            for (int j = 0; j < VEC; ++j) wsum += weight_of(fr.x[j], a, c);
          }
        } else {
          for (int col = c0 + lane; col < c1; col += 32) wsum += weight_of(load_elem(rowp, col), a, c);
        }
        wsum = warp_sum_u64(wsum);
        if (lane < VP_CS) st_peer_u64(peer_shared(&sh.xsum[cp][part], (uint32_t)lane), wsum);
        cluster_sync_all();
        // totals and the prefix in front of this sub-slice (parts are in column order)
        unsigned long long total = 0, before = 0;
        for (int q = lane; q < VP_PARTS; q += 32) {
          const unsigned long long v = sh.xsum[cp][q];
          total += v;
          before += q < part ? v : 0ull;
        }
        total = warp_sum_u64(total);
        before = warp_sum_u64(before);
        uint32_t rnd[4];
        philox4x32_10((uint32_t)cur, (uint32_t)b, 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), rnd);
        const unsigned long long R = (unsigned long long)rnd[0] | ((unsigned long long)rnd[1] << 32);
        const unsigned long long theta = __umul64hi(R, total);
        if (theta >= before && theta < before + wsum) {  // this sub-slice holds the threshold (exactly one does)
          // consecutive runs of columns per lane, then a scan over the lanes, then the token inside one run
          const int len = c1 - c0, per = (len + 31) / 32;
          const int t0 = c0 + lane * per, t1 = min(t0 + per, c1);
          unsigned long long lsum = 0;
          for (int col = t0; col < t1; ++col) lsum += weight_of(load_elem(rowp, col), a, c);
          unsigned long long inc = lsum;
#pragma unroll
          for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long up = __shfl_up_sync(FULL, inc, d);
            if (lane >= d) inc += up;
          }
          const unsigned long long rel = theta - before;
          const unsigned hit = __ballot_sync(FULL, inc > rel);
          const int l = hit ? __ffs(hit) - 1 : 31;
          int ans = 0;
          if (lane == l) {
            unsigned long long run = inc - lsum;
            ans = t1 - 1;
            for (int col = t0; col < t1; ++col) {
              run += weight_of(load_elem(rowp, col), a, c);
              if (run > rel) { ans = col; break; }
            }
            ans = ans < 0 ? 0 : (ans >= V ? V - 1 : ans);
          }
          ans = __shfl_sync(FULL, ans, l);
          if (lane < VP_CS) st_peer_s32(peer_shared(&sh.xpick[cp], (uint32_t)lane), ans);
        }
        cluster_sync_all();
        x = sh.xpick[cp];
      }
    }

    // ---- every warp of the cluster advances the walk by the step's pick (identical everywhere)
    int child = -1;
    for (int cc = 1; cc < n_nodes && child < 0; cc += 32) {
      const int c = cc + lane;
      const bool match = c < n_nodes && sh.par[c] == cur && sh.tok[c] == x;
      const unsigned mm = __ballot_sync(FULL, match);
      if (mm) child = cc + __ffs(mm) - 1;
    }
    const bool stop = child < 0 || acc == L;
    bits_all |= bits;
    if (writer) {
      out.out_tokens[(int64_t)b * (L + 1) + acc] = x;
      if (node_pick) node_pick[o + cur] = x;
      if (stop) { out.bonus_token[b] = x; out.accepted_len[b] = acc; }
      else out.accepted_nodes[(int64_t)b * (L + 1) + acc + 1] = child;
    }
    if (stop) break;
    cur = child;
    ++acc;
  }
  if (writer && status) status[b] = bits_all;
  cluster_sync_all();  // no CTA leaves while another may still write into its shared memory
}

// ------------------------------------------------------------------------------------ host side
size_t verify_path_workspace_bytes(int, int, int) { return 0; }  // the exchange lives in shared memory

template <typename T, int MODE>
static cudaError_t launch_verify_path_t(const ubt_tree& tree, const void* logits, int V, uint64_t seed, float temperature,
                                        int32_t* node_pick, const ubt_verify_result& out, int32_t* status,
                                        cudaStream_t st) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)tree.B * VP_CS);
  cfg.blockDim = dim3(VP_T);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;  // eight CTAs per sequence, resident together
  attr[0].val.clusterDim.x = VP_CS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_verify_path<T, MODE>, tree, static_cast<const T*>(logits), V, seed, temperature,
                            out, node_pick, status);
}

cudaError_t launch_verify_path(const ubt_tree& tree, const void* logits, int dtype, int V, int mode, uint64_t seed,
                               float temperature, void* ws, int32_t* node_pick, const ubt_verify_result& out,
                               int32_t* status, cudaStream_t st) {
  (void)ws;
  if (tree.B == 0) return cudaSuccess;
  if (dtype == UBT_BF16) {
    return mode == UBT_VERIFY_GREEDY
               ? launch_verify_path_t<__nv_bfloat16, UBT_VERIFY_GREEDY>(tree, logits, V, seed, temperature, node_pick, out, status, st)
               : launch_verify_path_t<__nv_bfloat16, UBT_VERIFY_SAMPLE>(tree, logits, V, seed, temperature, node_pick, out, status, st);
  }
  return mode == UBT_VERIFY_GREEDY
             ? launch_verify_path_t<float, UBT_VERIFY_GREEDY>(tree, logits, V, seed, temperature, node_pick, out, status, st)
             : launch_verify_path_t<float, UBT_VERIFY_SAMPLE>(tree, logits, V, seed, temperature, node_pick, out, status, st);
}

int verify_path_max_batch() { return (1 << 28) / VP_CS; }

cudaError_t ring_timeouts_path(unsigned int* out) { *out = 0; return cudaSuccess; }  // this file has no bounded waits

}  // namespace ubt
