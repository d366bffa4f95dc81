// Step a1: per-position vocabulary log-sum-exp and top-k candidates (eq. 3, "Candidate Sets").
//
// The rows*V logits are cut into equal contiguous spans, one per CTA, so that every SM streams the
// same number of bytes whatever rows is.  A span meets a few row segments; for each the CTA emits a
// partial (max, sum exp, sorted top-k) and a small merge kernel combines the partials of a row.
//
// Streaming one segment (k_lse_topk_ring, rows made of whole 16-byte fragments): chunks of the span arrive in a
// shared-memory ring through bulk asynchronous copies; every thread sums 2^((x - ref) log2 e) relative to a
// reference of its own and keeps the maximum of its fragments per chunk.  The candidates are found when the
// segment has streamed past: the k-th largest per-thread maximum bounds the k-th largest element from below, the
// few (thread, chunk) groups whose maximum reaches the bound are read again from L2, and their elements above
// the bound are ranked once as 64-bit (value, ~column) keys.  k_lse_topk is the plain-load form for other
// vocabularies (online max per thread, columns in a pool that is ranked whenever it fills, the next tile
// prefetched into registers).
#include "ubt_internal.h"
#include "ubt_merge.cuh"
#include "ubt_ring.cuh"

namespace ubt {

constexpr int G1_T = 512;    // threads per CTA
constexpr int G1_U = 2;      // 16-byte fragments per thread per tile
constexpr int G1_RC = 1024;  // pool entries ranked by counting; larger pools use k extraction rounds
constexpr int G1_SLACK = 4 * kMaxK;  // a tile starts with fewer pool entries than this

template <typename T, int VEC> struct RawFrag { uint4 v; };
template <typename T> struct RawFrag<T, 1> { float v; };

struct G1Shared {
  int cnt;     // pool entries
  int ntop;    // entries of top[]
  float taux;  // exclusive threshold: x enters the pool iff x > taux
  int pad;
  float redf[2 * (G1_T / 32)];
  unsigned long long red64[G1_T / 32];
  unsigned long long top[kMaxK];
  unsigned long long topn[kMaxK];
  unsigned long long keys[G1_RC + kMaxK];
};

template <typename T, int VEC>
__device__ __forceinline__ void load_frag(const T* seg, int nfrag, int i, RawFrag<T, VEC>& r) {
  if constexpr (VEC == 1) {
    r.v = i < nfrag ? load_elem(seg, i) : -INFINITY;
  } else {
    if (i < nfrag) {
      r.v = ldg_stream(reinterpret_cast<const uint4*>(seg) + i);
    } else {
      const uint32_t ninf = sizeof(T) == 2 ? 0xff80ff80u : 0xff800000u;
      r.v = make_uint4(ninf, ninf, ninf, ninf);
    }
  }
}

template <typename T, int VEC>
__device__ __forceinline__ void unpack_frag(const RawFrag<T, VEC>& r, float (&x)[VEC]) {
  if constexpr (VEC == 1) {
    x[0] = r.v;
  } else {
    Frag<T> f;
    f.unpack(r.v);
#pragma unroll
    for (int j = 0; j < VEC; ++j) x[j] = f.x[j];
  }
}

__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long v, unsigned long long* red) {
  v = warp_max_u64(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long r = 0;
  for (int w = 0; w < (int)(blockDim.x >> 5); ++w) r = red[w] > r ? red[w] : r;
  return r;
}

// Rank the pool (and the carried top list) exactly; afterwards top[0..ntop) is sorted best first,
// the pool is empty and, when k entries exist, taux is the k-th best value (strict from then on:
// a later element equal to it has a larger column than every kept entry).
template <typename T, int THREADS>
__device__ void flush_pool(G1Shared& sh, Span<int> pool, const T* rowp_raw, int V, int k) {
  const int tid = threadIdx.x;
  const Span<const T> rowp(rowp_raw, V, 303);
  const Span<unsigned long long> keys(sh.keys, G1_RC + kMaxK, 304), top(sh.top, kMaxK, 305), topn(sh.topn, kMaxK, 306);
  const int M = sh.cnt, nt = sh.ntop, total = M + nt;
  const int newn = total < k ? total : k;
  if (M <= G1_RC) {
    for (int i = tid; i < M; i += THREADS) {
      int col = pool[i];
      keys[i] = make_key(load_elem(rowp.ptr(col, 1), 0), col);
    }
    for (int i = tid; i < nt; i += THREADS) keys[M + i] = top[i];
    __syncthreads();
    for (int i = tid; i < total; i += THREADS) {
      unsigned long long ki = keys[i];
      int rank = 0;
      for (int j = 0; j < total; ++j) rank += keys[j] > ki;
      if (rank < k) topn[rank] = ki;
    }
  } else {
    unsigned long long last = ~0ull;
    for (int r = 0; r < newn; ++r) {
      unsigned long long best = 0;
      for (int i = tid; i < M; i += THREADS) {
        int col = pool[i];
        unsigned long long key = make_key(load_elem(rowp.ptr(col, 1), 0), col);
        if (key < last && key > best) best = key;
      }
      for (int i = tid; i < nt; i += THREADS) {
        unsigned long long key = top[i];
        if (key < last && key > best) best = key;
      }
      best = block_max_u64(best, sh.red64);
      if (tid == 0) topn[r] = best;
      last = best;
    }
  }
  __syncthreads();
  if (tid < newn) top[tid] = topn[tid];
  if (tid == 0) {
    sh.ntop = newn;
    sh.cnt = 0;
    if (newn == k) sh.taux = key_val(topn[k - 1]);
  }
  __syncthreads();
}

template <typename T, int VEC>
__global__ void __launch_bounds__(G1_T, VEC == 1 ? 1 : 2)
k_lse_topk(const T* __restrict__ logits, int64_t total, int V, int k, SpanPlan plan,
           float* __restrict__ part_ms, float* __restrict__ part_val, int32_t* __restrict__ part_idx,
           int32_t* __restrict__ part_cnt) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  G1Shared& sh = *reinterpret_cast<G1Shared*>(smem_raw);
  constexpr int TILE_FRAGS = G1_T * G1_U;
  const Span<int> pool(reinterpret_cast<int*>(smem_raw + sizeof(G1Shared)), TILE_FRAGS * VEC + G1_SLACK, 301);
  const long long nslots = (total / V) * plan.smax;
  const Span<float> g_ms(part_ms, nslots * 2, 311), g_val(part_val, nslots * k, 312);
  const Span<int32_t> g_idx(part_idx, nslots * k, 313), g_cnt(part_cnt, nslots, 314);
  const Span<const T> g_logits(logits, total, 302);

  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t lo = (int64_t)blockIdx.x * plan.span;
  const int64_t hi = lo + plan.span < total ? lo + plan.span : total;

  for (int64_t e = lo; e < hi;) {
    const int64_t row = e / V;
    const int c0 = (int)(e - row * V);
    const int c1 = (int)((int64_t)V - c0 < hi - e ? V : c0 + (hi - e));
    const T* rowp = g_logits.ptr(row * V, V);
    const T* seg = g_logits.ptr(row * V + c0, c1 - c0);
    const int nfrag = (c1 - c0) / VEC;  // spans and V are multiples of VEC on this path
    e += c1 - c0;

    if (tid == 0) { sh.cnt = 0; sh.ntop = 0; sh.taux = -INFINITY; }

    // Running (max, sum) start at a finite floor so that -inf padding gives exp2(-inf) = 0, never inf - inf.
    float m_t = -1.0e30f, s_t = 0.f, negml = 1.0e30f * kLog2e;
    RawFrag<T, VEC> cur[G1_U], nxt[G1_U];
#pragma unroll
    for (int u = 0; u < G1_U; ++u) load_frag<T, VEC>(seg, nfrag, u * G1_T + tid, cur[u]);

    // Bound for the k-th largest element from the per-thread maxima of the first tile: bisect the
    // top 16 key bits with CTA-wide counts; the result never exceeds the k-th largest maximum.
    {
      float tmax = -INFINITY;
      bool has = false;
#pragma unroll
      for (int u = 0; u < G1_U; ++u) {
        float x[VEC];
        unpack_frag<T, VEC>(cur[u], x);
#pragma unroll
        for (int j = 0; j < VEC; ++j) tmax = fmaxf(tmax, x[j]);
        has = has || (u * G1_T + tid < nfrag);
      }
      const uint32_t mykey = has ? f2key(tmax) : 0u;
      uint32_t lob = 0;
      for (int bit = 31; bit >= 16; --bit) {
        uint32_t cand = lob | (1u << bit);
        if (__syncthreads_count(mykey >= cand) >= k) lob = cand;
      }
      if (tid == 0 && lob != 0) {
        uint32_t below = lob - 1;
        if (below == 0x7fffffffu) below = 0x7ffffffeu;  // skip -0: it equals +0
        float t = key2f(below);
        sh.taux = (t != t) ? -INFINITY : t;
      }
      __syncthreads();
    }

    for (int base = 0; base < nfrag; base += TILE_FRAGS) {
      const float taux = sh.taux;
      if (base + TILE_FRAGS < nfrag) {
#pragma unroll
        for (int u = 0; u < G1_U; ++u)
          load_frag<T, VEC>(seg, nfrag, base + TILE_FRAGS + u * G1_T + tid, nxt[u]);
      }
#pragma unroll
      for (int u = 0; u < G1_U; ++u) {
        float x[VEC];
        unpack_frag<T, VEC>(cur[u], x);
        float vmax = x[0];
#pragma unroll
        for (int j = 1; j < VEC; ++j) vmax = fmaxf(vmax, x[j]);
        if (vmax > m_t) {  // online rescale; rare after the first fragments
          s_t *= ex2_approx(fmaf(m_t, kLog2e, -vmax * kLog2e));
          m_t = vmax;
          negml = -vmax * kLog2e;
        }
#pragma unroll
        for (int j = 0; j < VEC; ++j) s_t += ex2_approx(fmaf(x[j], kLog2e, negml));
        if (__any_sync(FULL, vmax > taux)) {
          const int col0 = c0 + (base + u * G1_T + tid) * VEC;
#pragma unroll
          for (int j = 0; j < VEC; ++j) {
            const bool hit = x[j] > taux;
            const unsigned mask = __ballot_sync(FULL, hit);
            if (mask) {
              const int leader = __ffs(mask) - 1;
              int at = 0;
              if (lane == leader) at = atomicAdd(&sh.cnt, __popc(mask));
              at = __shfl_sync(FULL, at, leader);
              if (hit) pool[at + __popc(mask & ((1u << lane) - 1))] = col0 + j;
            }
          }
        }
      }
#pragma unroll
      for (int u = 0; u < G1_U; ++u) cur[u] = nxt[u];
      // One barrier that also takes the decision: a warp may not re-read the counter after the barrier,
      // because faster warps are already appending hits of the next tile.  The last warp to arrive has
      // seen every append of this tile and counts only grow, so the OR is the decision on the final count.
      if (__syncthreads_or(*reinterpret_cast<volatile int*>(&sh.cnt) >= 4 * k))
        flush_pool<T, G1_T>(sh, pool, rowp, V, k);  // tighten the threshold early
    }
    flush_pool<T, G1_T>(sh, pool, rowp, V, k);

    // partial (max, sum exp) of the segment
    float mw = m_t;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mw = fmaxf(mw, __shfl_xor_sync(FULL, mw, o));
    if (lane == 0) sh.redf[tid >> 5] = mw;
    __syncthreads();
    float M = sh.redf[0];
    for (int w = 1; w < G1_T / 32; ++w) M = fmaxf(M, sh.redf[w]);
    float sw = s_t * ex2_approx((m_t - M) * kLog2e);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sw += __shfl_xor_sync(FULL, sw, o);
    if (lane == 0) sh.redf[G1_T / 32 + (tid >> 5)] = sw;
    __syncthreads();

    const int64_t c_first = (row * (int64_t)V) / plan.span;
    const int64_t slot = row * plan.smax + ((int64_t)blockIdx.x - c_first);
    if (tid == 0) {
      float S = 0.f;
      for (int w = 0; w < G1_T / 32; ++w) S += sh.redf[G1_T / 32 + w];
      g_ms[slot * 2] = M;
      g_ms[slot * 2 + 1] = S;
      g_cnt[slot] = sh.ntop;
    }
    if (tid < sh.ntop) {
      g_val[slot * k + tid] = key_val(sh.top[tid]);
      g_idx[slot * k + tid] = key_idx(sh.top[tid]);
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------- ring-fed version
// The logits arrive through the bulk-copy ring (ubt_ring.cuh), three CTAs per SM.
//
// Log-sum-exp without a running maximum in the common path: every thread sums 2^((x - ref) log2 e) relative to a
// reference of its own, the largest element of the first group it sees; an element more than 60 above the
// reference (rare) moves the reference up and rescales the sum.
//
// Top-k with deferred candidates: the streaming loop touches no candidate at all.  Per chunk a thread keeps the
// maximum of its own fragments (8 slots of shared memory per thread, a chunk uses slot chunk % 8, stored rounded
// up to bf16); per segment it keeps the exact maximum of all its elements so far.
//   * The k-th largest of the 256 per-thread maxima is a lower bound of the k-th largest element (the maxima are
//     256 distinct elements), and it only grows as more of the segment is seen.  It is bisected on the leading
//     key bits with CTA-wide counts BEFORE the segment's last chunk is processed.
//   * A thread whose slot maximum reaches the bound holds a possible candidate in that (thread, chunk) group of 8
//     fragments; on ordinary rows about k + k^2 / 512 groups qualify.  The threads list their groups, and the CTA
//     copies the listed groups again from global memory (L2) into a side buffer with asynchronous 16-byte
//     copies, 32 groups per round, one fragment per thread; the copies of the last round stay in flight while
//     the last chunk streams through the arithmetic (a load takes microseconds while every SM is streaming).
//   * After the last chunk every thread whose maximum of that chunk reaches the bound scans its fragments of it
//     once more in the stage, the side buffer is scanned, and the pool of (value, ~column) keys is ranked once.
// A pool that overflows (a row with hundreds of elements equal to its maximum) is handled by walking the segment
// again in column order, ranking after each step that produced a hit.
constexpr int G1R_T = 256, G1R_STAGES = 2, G1R_STAGE_BYTES = 32768, G1R_CTAS = 3;
constexpr int G1R_GROUP = 4;                                     // fragments per thread and loop iteration
constexpr int G1R_CHUNK_FRAGS = G1R_STAGE_BYTES / 16 / G1R_T;    // fragments of a full chunk per thread
constexpr int G1R_SLOTS = 8;                                     // chunk maxima a thread keeps
constexpr int G1R_POOL = 192;                                    // candidate pool entries
constexpr int G1R_ROUND = G1R_T / G1R_CHUNK_FRAGS;               // groups the CTA copies per round
constexpr int G1R_ITEMS = 128;  // groups a segment may list; more send it down the slow path

struct alignas(16) G1RShared {
  int cnt;     // pool entries (may exceed G1R_POOL: the surplus is dropped and the segment walked again)
  int ntop;    // entries of top[]
  float taux;  // slow path: exclusive threshold, x enters the pool iff x > taux
  int fail;    // a bounded wait gave up
  int nlist;   // entries of list[] (may exceed G1R_ITEMS)
  int pad[3];
  float redf[2 * (G1R_T / 32)];
  unsigned long long top[kMaxK];
  unsigned long long topn[kMaxK];
  unsigned long long pool[G1R_POOL];
  unsigned short gmax[G1R_SLOTS * G1R_T];  // [slot][thread] chunk maxima, bf16 bits rounded up
  uint4 side[G1R_T];                        // fragments read again, one per thread
  unsigned short list[G1R_ITEMS];           // thread << 8 | chunk of the groups to read again
};
static_assert(offsetof(G1RShared, side) % 16 == 0, "the side buffer receives 16-byte copies");
// three CTAs per SM: ring + this struct + the static barriers + 1 KiB the system reserves, times three, in 228 KiB
static_assert(G1R_CTAS * (G1R_STAGES * G1R_STAGE_BYTES + sizeof(G1RShared) + 128 + 1024) <= 233472, "three CTAs per SM");

__device__ __forceinline__ unsigned short bf16_bits_round_up(float x) {
  const uint32_t u = __float_as_uint(x);
  uint32_t h = u >> 16;
  if (!(u >> 31) && (u & 0xffffu)) h += 1;  // positive: magnitude up; negative: truncation already rounds up
  return (unsigned short)h;
}
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
               : "memory");
}
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Returns the number of elements appended (or dropped because the pool was full).
template <int VEC>
__device__ __forceinline__ int append_hits(G1RShared& sh, const float (&x)[VEC], float taux, int col0) {
  int hits = 0;
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    if (x[j] > taux) {
      const int at = atomicAdd(&sh.cnt, 1);
      if (at < G1R_POOL) sh.pool[at] = make_key(x[j], col0 + j);
      ++hits;
    }
  }
  return hits;
}

// Rank pool + carried list exactly (keys are unique); afterwards top[0..ntop) is sorted best first, the
// pool is empty and, when k entries exist, taux is the k-th best value (strict from then on).
__device__ void flush_keyed(G1RShared& sh, int k) {
  const int tid = threadIdx.x;
  const int M = sh.cnt < G1R_POOL ? sh.cnt : G1R_POOL, nt = sh.ntop, total = M + nt;
  const int newn = total < k ? total : k;
  for (int i = tid; i < total; i += G1R_T) {
    const unsigned long long ki = i < M ? sh.pool[i] : sh.top[i - M];
    int rank = 0;
    for (int j = 0; j < M; ++j) rank += sh.pool[j] > ki;
    for (int j = 0; j < nt; ++j) rank += sh.top[j] > ki;
    if (rank < k) sh.topn[rank] = ki;
  }
  __syncthreads();
  if (tid < newn) sh.top[tid] = sh.topn[tid];
  if (tid == 0) {
    sh.ntop = newn;
    sh.cnt = 0;
    if (newn == k) sh.taux = key_val(sh.topn[k - 1]);
  }
  __syncthreads();
}

template <typename T>
__global__ void __launch_bounds__(G1R_T, G1R_CTAS)
k_lse_topk_ring(const T* __restrict__ logits, int64_t total, int V, int k, SpanPlan plan,
                 float* __restrict__ part_ms, float* __restrict__ part_val, int32_t* __restrict__ part_idx,
                 int32_t* __restrict__ part_cnt) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int STAGE_ELEMS = G1R_STAGE_BYTES / (int)sizeof(T);
  constexpr int CHUNK_FRAGS = G1R_CHUNK_FRAGS;
  constexpr int RING_BYTES = G1R_STAGES * G1R_STAGE_BYTES;
  constexpr int NW = G1R_T / 32;
  constexpr int LOW_BIT = sizeof(T) == 2 ? 16 : 12;  // bf16 values have no key bits below 16
  unsigned char* ring = smem_raw;
  G1RShared& sh = *reinterpret_cast<G1RShared*>(smem_raw + RING_BYTES);
  unsigned short* gmax = sh.gmax;
  __shared__ uint64_t full[G1R_STAGES];

  const int tid = threadIdx.x, lane = tid & 31;
  uint4* side = sh.side + tid;
  unsigned short* list = sh.list;
  int* nlist = &sh.nlist;
  const int64_t lo = (int64_t)blockIdx.x * plan.span;
  const int64_t hi = lo + plan.span < total ? lo + plan.span : total;
  pdl_wait();  // nothing is read or written before the kernel in front has completed
  pdl_launch_dependents();
  if (lo >= hi) return;
  const long long nslots = (total / V) * plan.smax;
  const Span<float> g_ms(part_ms, nslots * 2, 341), g_val(part_val, nslots * k, 342);
  const Span<int32_t> g_idx(part_idx, nslots * k, 343), g_cnt(part_cnt, nslots, 344);

  if (tid == 0) {
    for (int s = 0; s < G1R_STAGES; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    sh.fail = 0;
  }
  __syncthreads();
  RingProducer<T, G1R_STAGES, G1R_STAGE_BYTES> prod;
  if (tid == 0) {
    prod.init(lo, hi, V);
    for (int i = 0; i < G1R_STAGES - 1; ++i) prod.issue_one(logits, ring, full);
  }
  RingPos<G1R_STAGES> rp;
  rp.init();
  int consumed = 0;
  bool failed = false;
  bool ahead = false;  // the copy that the next chunk would issue is already on its way
  const unsigned long long l2e2 = pack2(kLog2e, kLog2e);

  for (int64_t pos = lo; pos < hi && !failed;) {
    Segment sg;
    sg.at(pos, hi, V);
    const T* seg = logits + sg.row * (int64_t)V + sg.col0;
    if (tid == 0) { sh.cnt = 0; sh.ntop = 0; sh.taux = -INFINITY; *nlist = 0; }
    float ref = -1.0e30f, negref = 1.0e30f * kLog2e;  // ref = -1e30: not fixed yet
    float segmax = -INFINITY;
    float taux = -INFINITY;  // exclusive bound: an element is a candidate iff it is > taux
    int side_col = -1;       // column of the fragment this lane has in flight to the side buffer
    unsigned long long acc[G1R_GROUP];  // packed pairs of partial sums (one FADD2 adds two exponentials)
#pragma unroll
    for (int u = 0; u < G1R_GROUP; ++u) acc[u] = 0ull;

    // the bound from the per-thread maxima seen so far
    auto bisect = [&]() {
      const uint32_t mykey = segmax > -INFINITY ? f2key(segmax) : 0u;
      uint32_t lob = 0;
      for (int bit = 31; bit >= LOW_BIT; --bit) {
        const uint32_t cand = lob | (1u << bit);
        if (__syncthreads_count(mykey >= cand) >= k) lob = cand;
      }
      if (lob != 0u) {
        uint32_t below = lob - 1;
        if (below == 0x7fffffffu) below = 0x7ffffffeu;  // skip -0: it equals +0
        const float t = key2f(below), t0 = key2f(lob);
        if (t == t && t0 == t0) taux = t;
      }
    };
    // what this thread copied to the side buffer
    auto scan_side = [&]() {
      cp_async_wait();
      if (side_col >= 0) {
        Frag<T> fr;
        fr.unpack(*side);
        append_hits<VEC>(sh, fr.x, taux, side_col);
      }
      side_col = -1;
    };

    int chunk = 0;
    for (int c = 0; c < sg.len; c += STAGE_ELEMS, ++chunk) {
      const int l = sg.len - c < STAGE_ELEMS ? sg.len - c : STAGE_ELEMS;
      const bool last = c + STAGE_ELEMS >= sg.len;
      if (*reinterpret_cast<volatile int*>(&sh.fail)) { failed = true; break; }
      if (tid == 0 && !ahead) prod.issue_one(logits, ring, full);
      ahead = false;
      if (last && chunk > 0) {
        // the chunks before the last: bound, then the groups that may hold a candidate, read again
        bisect();
#pragma unroll
        for (int slot = 0; slot < G1R_SLOTS; ++slot) {
          if (slot < chunk && __uint_as_float((uint32_t)gmax[slot * G1R_T + tid] << 16) > taux) {
            for (int ch = slot; ch < chunk; ch += G1R_SLOTS) {
              const int at = atomicAdd(nlist, 1);
              if (at < G1R_ITEMS && ch < 256) list[at] = (unsigned short)((tid << 8) | ch);
              else atomicAdd(&sh.cnt, G1R_POOL + 1);  // the list is full: this segment takes the slow path
            }
          }
        }
        __syncthreads();
        const int n_items = *nlist < G1R_ITEMS ? *nlist : G1R_ITEMS;
        for (int i0 = 0; i0 < n_items; i0 += G1R_ROUND) {
          const int it = i0 + tid / CHUNK_FRAGS;
          if (it < n_items) {
            const int owner = list[it] >> 8, cc = (list[it] & 255) * STAGE_ELEMS;
            const int f = (tid % CHUNK_FRAGS) * G1R_T + owner;  // a chunk before the last is full
            cp_async_16(side, reinterpret_cast<const uint4*>(seg + cc) + f);
            side_col = sg.col0 + cc + f * VEC;
          }
          if (i0 + G1R_ROUND < n_items) scan_side();  // more rounds follow: take this one in first
        }
      }
      const bool ok = mbar_wait(&full[rp.stage], rp.parity);
      if (!ok) sh.fail = 1;
      const uint4* stage = reinterpret_cast<const uint4*>(ring + (size_t)rp.stage * G1R_STAGE_BYTES) + tid;
      const int nfrag = ok ? l / VEC : 0;
      float cmax = -INFINITY;
      int f0 = 0;
      for (; f0 + G1R_GROUP * G1R_T <= nfrag; f0 += G1R_GROUP * G1R_T) {  // full groups: no bounds checks
        float x[G1R_GROUP][VEC];
        float vmax[G1R_GROUP];
#pragma unroll
        for (int u = 0; u < G1R_GROUP; ++u) {
          Frag<T> fr;
          fr.unpack(stage[f0 + u * G1R_T]);
          vmax[u] = fr.x[0];
#pragma unroll
          for (int j = 0; j < VEC; ++j) { x[u][j] = fr.x[j]; vmax[u] = fmaxf(vmax[u], fr.x[j]); }
        }
        const float gm = fmaxf(fmaxf(vmax[0], vmax[1]), fmaxf(vmax[2], vmax[3]));
        cmax = fmaxf(cmax, gm);
        if (gm > ref + 60.f) {  // rare: the first elements of a segment, or an element far above the reference
          const float sc = ex2_approx(fmaf(ref, kLog2e, -gm * kLog2e));
#pragma unroll
          for (int u = 0; u < G1R_GROUP; ++u) acc[u] = fma2(acc[u], pack2(sc, sc), 0ull);
          ref = gm;
          negref = -gm * kLog2e;
        }
#pragma unroll
        for (int u = 0; u < G1R_GROUP; ++u) {
#pragma unroll
          for (int j = 0; j < VEC; j += 2) {
            float y0, y1;
            unpack2(fma2(pack2(x[u][j], x[u][j + 1]), l2e2, pack2(negref, negref)), y0, y1);
            acc[u] = add2(acc[u], pack2(ex2_approx(y0), ex2_approx(y1)));
          }
        }
      }
      for (; f0 + tid < nfrag; f0 += G1R_T) {  // ragged end of a chunk
        Frag<T> fr;
        fr.unpack(stage[f0]);
        float vm = fr.x[0];
#pragma unroll
        for (int j = 1; j < VEC; ++j) vm = fmaxf(vm, fr.x[j]);
        cmax = fmaxf(cmax, vm);
        if (vm > ref + 60.f) {
          const float sc = ex2_approx(fmaf(ref, kLog2e, -vm * kLog2e));
#pragma unroll
          for (int u = 0; u < G1R_GROUP; ++u) acc[u] = fma2(acc[u], pack2(sc, sc), 0ull);
          ref = vm;
          negref = -vm * kLog2e;
        }
#pragma unroll
        for (int j = 0; j < VEC; j += 2) {
          float y0, y1;
          unpack2(fma2(pack2(fr.x[j], fr.x[j + 1]), l2e2, pack2(negref, negref)), y0, y1);
          acc[0] = add2(acc[0], pack2(ex2_approx(y0), ex2_approx(y1)));
        }
      }
      segmax = fmaxf(segmax, cmax);
      if (!last) {
        const int slot = chunk & (G1R_SLOTS - 1);
        float m = cmax;
        if (chunk >= G1R_SLOTS) m = fmaxf(m, __uint_as_float((uint32_t)gmax[slot * G1R_T + tid] << 16));
        gmax[slot * G1R_T + tid] = bf16_bits_round_up(m);
      } else {
        // the last chunk is still in its stage: a thread whose maximum of it reaches the bound scans its fragments
        // once more (a segment of one chunk gets its bound only now)
        if (chunk == 0) bisect();
        if (cmax > taux) {
          for (int f = 0; f + tid < nfrag; f += G1R_T) {
            Frag<T> fr;
            fr.unpack(stage[f]);
            append_hits<VEC>(sh, fr.x, taux, sg.col0 + c + (f + tid) * VEC);
          }
        }
        scan_side();
      }
      __syncthreads();  // the stage is free for the copy after next; after the last chunk: the pool is complete
      rp.next();
      ++consumed;
    }
    if (failed) break;
    // the stage of the last chunk is free: keep the ring full while the candidates are ranked
    if (tid == 0) prod.issue_one(logits, ring, full);
    ahead = true;

    if (sh.cnt > G1R_POOL) {
      // more candidates than the pool holds: walk the segment in column order, 256 fragments at a time; once k
      // entries stand, only a strictly larger element can still enter (an equal one has the higher column)
      __syncthreads();
      if (tid == 0) { sh.cnt = 0; sh.ntop = 0; sh.taux = taux; }
      __syncthreads();
      constexpr int SLICE = G1R_POOL / VEC;  // fragments whose elements fit the pool in any case
      const int nfrag_seg = sg.len / VEC;
      for (int g0 = 0; g0 < nfrag_seg; g0 += G1R_T) {
        const float tx = sh.taux;
        const int f = g0 + tid;
        Frag<T> fr;
        int hits = 0;
        if (f < nfrag_seg) {
          fr.unpack(__ldg(reinterpret_cast<const uint4*>(seg) + f));
          hits = append_hits<VEC>(sh, fr.x, tx, sg.col0 + f * VEC);
        }
        if (!__syncthreads_or(hits > 0)) continue;
        if (sh.cnt <= G1R_POOL) {
          flush_keyed(sh, k);
          continue;
        }
        __syncthreads();  // too many for one ranking: the same fragments again, a pool's worth at a time
        if (tid == 0) sh.cnt = 0;
        __syncthreads();
        for (int s0 = 0; s0 < G1R_T; s0 += SLICE) {
          const float tx2 = sh.taux;
          int h2 = 0;
          if (f < nfrag_seg && tid >= s0 && tid < s0 + SLICE) h2 = append_hits<VEC>(sh, fr.x, tx2, sg.col0 + f * VEC);
          if (__syncthreads_or(h2 > 0)) flush_keyed(sh, k);
        }
      }
    } else {
      flush_keyed(sh, k);
    }

    // partial (max, sum exp) of the segment from the per-thread (reference, sum) pairs
    float s_t;
    {
      float a0, a1;
      unpack2(add2(add2(acc[0], acc[1]), add2(acc[2], acc[3])), a0, a1);
      s_t = a0 + a1;
    }
    float mw = ref;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mw = fmaxf(mw, __shfl_xor_sync(FULL, mw, o));
    if (lane == 0) sh.redf[tid >> 5] = mw;
    __syncthreads();
    float M = sh.redf[0];
    for (int w = 1; w < NW; ++w) M = fmaxf(M, sh.redf[w]);
    float sw = s_t * ex2_approx((ref - M) * kLog2e);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sw += __shfl_xor_sync(FULL, sw, o);
    if (lane == 0) sh.redf[NW + (tid >> 5)] = sw;
    __syncthreads();
    const int64_t c_first = (sg.row * (int64_t)V) / plan.span;
    const int64_t slot = sg.row * plan.smax + ((int64_t)blockIdx.x - c_first);
    if (tid == 0) {
      float S = 0.f;
      for (int w = 0; w < NW; ++w) S += sh.redf[NW + w];
      g_ms[slot * 2] = M;
      g_ms[slot * 2 + 1] = S;
      g_cnt[slot] = sh.ntop;
    }
    if (tid < sh.ntop) {
      g_val[slot * k + tid] = key_val(sh.top[tid]);
      g_idx[slot * k + tid] = key_idx(sh.top[tid]);
    }
    __syncthreads();
    pos += sg.len;
  }
  cp_async_wait();
  __syncthreads();
  if (tid == 0 && *reinterpret_cast<volatile int*>(&sh.fail)) {
    prod.drain(consumed > 0 ? consumed - 1 : 0, full);
    // a wait gave up: mark every segment of this span (written or not) so that the merge reports it
    for (int64_t pos = lo; pos < hi;) {
      Segment sg;
      sg.at(pos, hi, V);
      const int64_t c_first = (sg.row * (int64_t)V) / plan.span;
      g_cnt[sg.row * plan.smax + ((int64_t)blockIdx.x - c_first)] = -1;
      pos += sg.len;
    }
  }
}

// One warp per row: combine the partials of the row's segments (see merge_row_warp in ubt_merge.cuh).
__global__ void __launch_bounds__(128)
k_merge_topk(MergeParts parts, int64_t rows, int V, int k, int32_t* __restrict__ cand_ids,
             float* __restrict__ cand_lp) {
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  merge_row_warp(parts, rows, row, V, k, cand_ids, cand_lp, threadIdx.x & 31);
}

// One CTA per row, lists staged in shared memory (see merge_row_cta in ubt_merge.cuh).
constexpr int MERGE_CTA_T = 128;
__global__ void __launch_bounds__(MERGE_CTA_T)
k_merge_topk_cta(MergeSource src, int64_t rows, int V, int k, int32_t* __restrict__ cand_ids,
                 float* __restrict__ cand_lp, MergeShardOut so) {
  extern __shared__ __align__(16) unsigned char merge_smem[];
  const int lists = src.shards ? src.shards : src.parts.plan.smax;
  unsigned long long* s_key = reinterpret_cast<unsigned long long*>(merge_smem);
  int* s_cnt = reinterpret_cast<int*>(s_key + (size_t)lists * k);
  float* s_red = reinterpret_cast<float*>(s_cnt + lists);
  merge_row_cta<MERGE_CTA_T>(src, rows, blockIdx.x, V, k, cand_ids, cand_lp, so, s_key, s_cnt, s_red);
}

// ------------------------------------------------------------------------------------ host side
SpanPlan make_span_plan(int64_t rows, int V, int ctas, int64_t min_span) {
  SpanPlan p;
  const int64_t total = rows * (int64_t)V;
  int64_t span = (total + ctas - 1) / ctas;
  if (span < min_span) span = min_span;
  span = (span + 255) / 256 * 256;
  p.span = span;
  p.grid = (int)((total + span - 1) / span);
  if (p.grid < 1) p.grid = 1;
  p.smax = (int)(((int64_t)V + span - 1) / span) + 1;
  return p;
}

SpanPlan topk_plan(int64_t rows, int V) {
  return make_span_plan(rows, V, device_info().sm_count * G1R_CTAS, 32768);
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t topk_workspace_bytes(int64_t rows, int V, int k) {
  const SpanPlan p = topk_plan(rows, V);
  const size_t slots = (size_t)rows * p.smax;
  return align_up(slots * 2 * sizeof(float), 256) + align_up(slots * k * sizeof(float), 256) +
         align_up(slots * k * sizeof(int32_t), 256) + align_up(slots * sizeof(int32_t), 256);
}

TopkWorkspace carve_topk_workspace(void* ws, int64_t rows, int V, int k) {
  TopkWorkspace w;
  w.plan = topk_plan(rows, V);
  const size_t slots = (size_t)rows * w.plan.smax;
  unsigned char* p = static_cast<unsigned char*>(ws);
  w.part_ms = reinterpret_cast<float*>(p); p += align_up(slots * 2 * sizeof(float), 256);
  w.part_val = reinterpret_cast<float*>(p); p += align_up(slots * k * sizeof(float), 256);
  w.part_idx = reinterpret_cast<int32_t*>(p); p += align_up(slots * k * sizeof(int32_t), 256);
  w.part_cnt = reinterpret_cast<int32_t*>(p);
  return w;
}

template <typename T, int VEC>
static cudaError_t launch_lse_topk_t(const void* logits, int64_t rows, int V, int k,
                                     const TopkWorkspace& w, cudaStream_t st) {
  const size_t smem = sizeof(G1Shared) + sizeof(int) * (size_t)(G1_T * G1_U * VEC + G1_SLACK);
  auto kern = k_lse_topk<T, VEC>;
  cudaError_t e = allow_max_dynamic_smem<k_lse_topk<T, VEC>>();
  if (e != cudaSuccess) return e;
  kern<<<w.plan.grid, G1_T, smem, st>>>(static_cast<const T*>(logits), rows * (int64_t)V, V, k, w.plan,
                                        w.part_ms, w.part_val, w.part_idx, w.part_cnt);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_lse_topk_ring_t(const void* logits, int64_t rows, int V, int k, const TopkWorkspace& w,
                                          cudaStream_t st) {
  const size_t smem = (size_t)G1R_STAGES * G1R_STAGE_BYTES + sizeof(G1RShared);
  auto kern = k_lse_topk_ring<T>;
  cudaError_t e = allow_max_dynamic_smem<k_lse_topk_ring<T>>();
  if (e != cudaSuccess) return e;
  return launch_kernel(kern, dim3(w.plan.grid), dim3(G1R_T), smem, st, true, static_cast<const T*>(logits),
                       rows * (int64_t)V, V, k, w.plan, w.part_ms, w.part_val, w.part_idx, w.part_cnt);
}

cudaError_t launch_lse_topk(const void* logits, int dtype, int64_t rows, int V, int k,
                            const TopkWorkspace& w, cudaStream_t st) {
  // rows that are whole 16-byte fragments go through the bulk-copy ring; other V use plain scalar loads
  if (dtype == UBT_BF16) {
    if (V % 8 == 0) return launch_lse_topk_ring_t<__nv_bfloat16>(logits, rows, V, k, w, st);
    return launch_lse_topk_t<__nv_bfloat16, 1>(logits, rows, V, k, w, st);
  }
  if (V % 4 == 0) return launch_lse_topk_ring_t<float>(logits, rows, V, k, w, st);
  return launch_lse_topk_t<float, 1>(logits, rows, V, k, w, st);
}

static cudaError_t launch_merge_cta(const MergeSource& src, int64_t rows, int V, int k, int32_t* cand_ids,
                                    float* cand_lp, const MergeShardOut& so, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  const int lists = src.shards ? src.shards : src.parts.plan.smax;
  const size_t smem = (size_t)lists * k * 8 + (size_t)lists * 4 + 16;
  if (smem > (size_t)device_info().max_smem_optin) return cudaErrorNotSupported;
  cudaError_t e = allow_max_dynamic_smem<k_merge_topk_cta>();
  if (e != cudaSuccess) return e;
  k_merge_topk_cta<<<(unsigned)rows, MERGE_CTA_T, smem, st>>>(src, rows, V, k, cand_ids, cand_lp, so);
  return cudaGetLastError();
}

size_t shard_partial_bytes(int64_t rows, int k) {
  return align_up((size_t)rows * 2 * sizeof(float), 256) + 2 * align_up((size_t)rows * k * 4, 256) +
         align_up((size_t)rows * sizeof(int32_t), 256);
}
// The four arrays of one rank's partial: (max, sum exp) [rows,2], values [rows,k], ids [rows,k], counts [rows].
MergeShardOut carve_shard_partial(void* partial, int64_t rows, int k, int id_offset) {
  unsigned char* p = static_cast<unsigned char*>(partial);
  MergeShardOut so{};
  so.ms = reinterpret_cast<float*>(p); p += align_up((size_t)rows * 2 * sizeof(float), 256);
  so.val = reinterpret_cast<float*>(p); p += align_up((size_t)rows * k * 4, 256);
  so.idx = reinterpret_cast<int32_t*>(p); p += align_up((size_t)rows * k * 4, 256);
  so.cnt = reinterpret_cast<int32_t*>(p);
  so.id_offset = id_offset;
  return so;
}

cudaError_t launch_merge_topk_shard(int64_t rows, int V, int k, const TopkWorkspace& w, void* partial, int v0,
                                    cudaStream_t st) {
  const MergeSource src{merge_parts(w), 0, 0};
  return launch_merge_cta(src, rows, V, k, nullptr, nullptr, carve_shard_partial(partial, rows, k, v0), st);
}

cudaError_t launch_merge_shards(const void* gathered, int shards, int64_t rows, int k, int32_t* cand_ids,
                                float* cand_lp, cudaStream_t st) {
  const MergeShardOut a = carve_shard_partial(const_cast<void*>(gathered), rows, k, 0);
  MergeSource src{};
  src.parts = MergeParts{SpanPlan{}, a.ms, a.val, a.idx, a.cnt};
  src.shards = shards;
  src.shard_bytes = (int64_t)shard_partial_bytes(rows, k);
  return launch_merge_cta(src, rows, shards, k, cand_ids, cand_lp, MergeShardOut{}, st);
}

cudaError_t launch_merge_topk(int64_t rows, int V, int k, const TopkWorkspace& w, int32_t* cand_ids,
                              float* cand_lp, cudaStream_t st) {
  // many entries per row (large k): a CTA per row ranks them out of shared memory
  if ((int64_t)w.plan.smax * k > 64) {
    const MergeSource src{merge_parts(w), 0, 0};
    const cudaError_t e = launch_merge_cta(src, rows, V, k, cand_ids, cand_lp, MergeShardOut{}, st);
    if (e != cudaErrorNotSupported) return e;
  }
  const int warps = 4;
  const int grid = (int)((rows + warps - 1) / warps);
  k_merge_topk<<<grid, warps * 32, 0, st>>>(merge_parts(w), rows, V, k, cand_ids, cand_lp);
  return cudaGetLastError();
}

// Number of bounded waits that gave up in this file's kernels (0 in a healthy run).
cudaError_t ring_timeouts_topk(unsigned int* out) { return cudaMemcpyFromSymbol(out, g_ring_timeouts, sizeof *out); }

#ifdef UBT_BOUNDS_CHECK
// Debug builds only: first out-of-range index seen by the kernels of this file (flag, site, index, limit).
cudaError_t bounds_report_topk(long long out[4]) {
  BoundsReport r;
  cudaError_t e = cudaMemcpyFromSymbol(&r, g_bounds_report, sizeof r);
  out[0] = r.flag; out[1] = r.site; out[2] = r.index; out[3] = r.limit;
  return e;
}
#endif

}  // namespace ubt
