// Step a4: the target's pick at every tree slot, then the acceptance walk (Appendix A, verification).
//
// Greedy: B*N*V target logits are cut into equal contiguous spans, one per CTA; each CTA emits, for
// every row segment it meets, the (value, lowest token) maximum as one 64-bit key.  The walk kernel
// reduces a row's few keys, so no atomics and no zero-initialised scratch are needed.  Rows made of whole
// 16-byte fragments stream through a shared-memory ring fed by bulk asynchronous copies
// (k_row_argmax_ring); other vocabularies use the plain-load kernel k_row_argmax.
// Sampling: k_row_weights_ring passes over every row twice through the same kind of ring -- pass 1 finds the
// row maximum, pass 2 (partly served from L2) turns every logit into an integer weight with a fixed sequence
// of IEEE operations and sums them per 1024-token block -- and k_row_pick finds the block, then the token,
// that holds the row's Philox threshold.  Integer sums make the pick independent of the order of addition.
// k_row_sample is the plain-load form for other vocabularies.
// The V-wide kernels are launched programmatically, so their CTAs become resident behind the kernel in front of
// them; by default they wait there for that kernel to complete before they read anything (stream order).  Only
// when the caller opts in (ubt_verify_opts.early_start) do they stream at once and wait at their very end.
#include "ubt_internal.h"
#include "ubt_pick.cuh"
#include "ubt_ring.cuh"

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
    bool saw_nan = false;
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
        for (int j = 1; j < VEC; ++j) vmax = max_nan(vmax, x[j]);
        saw_nan = saw_nan || vmax != vmax;
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
    key = saw_nan ? kKeyNaNSeen : key;
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

// ---------------------------------------------------------------------------- greedy picks, ring-fed
// One CTA per SM; the span's chunks arrive through the shared-memory ring (ubt_ring.cuh).
//
// Only an element above everything seen earlier in the row can be the pick (ties go to the lower column,
// and earlier means lower column here), so each warp carries a threshold: the largest value seen by the CTA
// in earlier chunks (shared, read once per chunk) or by the warp in its earlier fragments.  The common case
// per 16-byte fragment is a packed maximum, one compare and one vote; a lane records (value, column) only
// when its fragment beats the threshold.  A threshold is never taken from the same chunk of another warp:
// that warp's element could sit at a higher column than an equal one of this warp.
template <typename T, int STAGES, int STAGE_BYTES, int THREADS, int CTAS>
__global__ void __launch_bounds__(THREADS, CTAS)
k_row_argmax_ring(const T* __restrict__ logits, int64_t total, int V, SpanPlan plan,
                  unsigned long long* __restrict__ part_key_, int early) {
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ uint64_t full[STAGES];
  __shared__ unsigned long long red[THREADS / 32];
  // Ordering key of the CTA's running maximum in this row segment (0 = none), double-buffered by chunk parity:
  // chunk t reads slot t&1 and publishes into slot (t+1)&1, so a slow warp never sees a value of its own chunk.
  __shared__ uint32_t s_thr[2];
  __shared__ int s_fail;  // set by a thread whose bounded wait gave up; read by all after the next barrier
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int STAGE_ELEMS = STAGE_BYTES / (int)sizeof(T);
  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t lo = (int64_t)blockIdx.x * plan.span;
  const int64_t hi = lo + plan.span < total ? lo + plan.span : total;
  const Span<unsigned long long> part_key(part_key_, (total / V) * plan.smax, 401);
  // Stream order is the default: nothing is read or written before the kernel in front on the stream has
  // completed.  With `early` (the caller vouches that the target logits were complete, and the scratch unused,
  // before that kernel's call was enqueued) the span is streamed at once and the wait moves to the very end.
  if (!early) pdl_wait();
  pdl_launch_dependents();  // the walk kernel may be scheduled; it waits for this grid before reading
  if (lo >= hi) {
    if (early && tid == 0) pdl_wait();
    return;
  }

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_thr[0] = s_thr[1] = 0u;
    s_fail = 0;
  }
  __syncthreads();
  RingProducer<T, STAGES, STAGE_BYTES> prod;
  if (tid == 0) {
    prod.init(lo, hi, V);
    for (int i = 0; i < STAGES - 1; ++i) prod.issue_one(logits, ring, full);
  }
  RingPos<STAGES> rp;
  rp.init();
  int consumed = 0;  // chunks fully processed (indexes the threshold slots and, after a failure, the drain)
  bool failed = false;
  for (int64_t pos = lo; pos < hi && !failed;) {
    Segment sg;
    sg.at(pos, hi, V);
    float best = -INFINITY, wthr = -INFINITY;  // wthr: warp-uniform threshold, -inf = none yet
    int bcol = -1;
    bool saw_nan = false;
    // One fragment against the threshold; every lane of the warp must call it (it votes).
    auto visit = [&](const uint4& v, float fm, int col) {
      const bool beat = fm > wthr;
      saw_nan = saw_nan || fm != fm;
      if (__any_sync(FULL, beat)) {
        if (beat) {
          Frag<T> x;
          x.unpack(v);
          int j0 = 0;
#pragma unroll
          for (int j = VEC - 1; j >= 0; --j) j0 = x.x[j] == fm ? j : j0;  // first element equal to the maximum
          best = fm;
          bcol = col + j0;
        }
        const uint32_t mk = __reduce_max_sync(FULL, beat ? f2key(fm) : 0u);
        wthr = fmaxf(wthr, key2f(mk));
      }
    };
    for (int c = 0; c < sg.len; c += STAGE_ELEMS) {
      const int l = sg.len - c < STAGE_ELEMS ? sg.len - c : STAGE_ELEMS;
      const uint32_t tk = s_thr[consumed & 1];  // published before the previous barrier
      if (*reinterpret_cast<volatile int*>(&s_fail)) { failed = true; break; }  // same answer for every thread
      if (tid == 0) prod.issue_one(logits, ring, full);  // into the stage freed by the previous barrier
      if (tk != 0u) wthr = fmaxf(wthr, key2f(tk));
      if (mbar_wait(&full[rp.stage], rp.parity)) {
        const uint4* stage = reinterpret_cast<const uint4*>(ring + (size_t)rp.stage * STAGE_BYTES) + tid;
        const int nfrag = l / VEC;
        const int colbase = sg.col0 + c + tid * VEC;
        int f0 = 0;
        for (; f0 + 4 * THREADS <= nfrag; f0 += 4 * THREADS) {  // four fragments per vote
          uint4 v[4];
          float fm[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) v[u] = stage[f0 + u * THREADS];
#pragma unroll
          for (int u = 0; u < 4; ++u) fm[u] = frag_max(v[u], (const T*)nullptr);
          if (__any_sync(FULL, !(max_nan(max_nan(fm[0], fm[1]), max_nan(fm[2], fm[3])) <= wthr))) {
#pragma unroll
            for (int u = 0; u < 4; ++u) visit(v[u], fm[u], colbase + (f0 + u * THREADS) * VEC);
          }
        }
        for (; f0 < nfrag; f0 += THREADS) {  // ragged end of a chunk; the trip count is warp-uniform
          uint4 v = make_uint4(0, 0, 0, 0);
          float fm = -INFINITY;
          if (f0 + tid < nfrag) { v = stage[f0]; fm = frag_max(v, (const T*)nullptr); }
          visit(v, fm, colbase + f0 * VEC);
        }
        if (lane == 0 && wthr > -INFINITY) atomicMax(&s_thr[(consumed + 1) & 1], f2key(wthr));
      } else {
        s_fail = 1;
      }
      __syncthreads();  // frees the stage; makes the thresholds and a possible failure visible
      rp.next();
      ++consumed;
    }
    if (failed) break;
    unsigned long long key = bcol >= 0 ? make_key(best, bcol) : 0ull;
    key = saw_nan ? kKeyNaNSeen : key;
    key = warp_max_u64(key);
    if (lane == 0) red[tid >> 5] = key;
    if (tid == 0) s_thr[0] = s_thr[1] = 0u;  // nobody touches them between the two barriers
    __syncthreads();
    if (tid == 0) {
      unsigned long long r = red[0];
      for (int w = 1; w < THREADS / 32; ++w) r = red[w] > r ? red[w] : r;
      const int64_t c_first = (sg.row * (int64_t)V) / plan.span;
      part_key[sg.row * plan.smax + ((int64_t)blockIdx.x - c_first)] = r;
    }
    pos += sg.len;
  }
  __syncthreads();
  if (tid == 0 && *reinterpret_cast<volatile int*>(&s_fail)) {
    prod.drain(consumed > 0 ? consumed - 1 : 0, full);
    for (int64_t pos = lo; pos < hi;) {  // a wait gave up: mark every segment of this span for the walk
      Segment sg;
      sg.at(pos, hi, V);
      const int64_t c_first = (sg.row * (int64_t)V) / plan.span;
      part_key[sg.row * plan.smax + ((int64_t)blockIdx.x - c_first)] = kKeyGaveUp;
      pos += sg.len;
    }
  }
  // An early start must not become an early finish: the walk behind this kernel waits for THIS grid only, so
  // this grid may not complete before the kernel in front of it (the tree builder) has.
  if (early && tid == 0) pdl_wait();
}

// ---------------------------------------------------------------------------- sampling picks
// Two weights at once with the packed fp32 instructions of sm_100 (fma/add .f32x2): the same IEEE operations
// per component as weight_of, half the issue slots for the arithmetic part.
struct WeightConsts2 {  // the routine's constants, duplicated into both halves
  // The polynomial's coefficients carry the factor 2^40 of the weight: scaling every Horner step by a power of
  // two changes no rounding, so the mantissa bits are those of weight_of and the exponent insert is one add.
  unsigned long long a, c, big, nbig, none, c5, c4, c3, c2, c1, c0;
  __device__ __forceinline__ void init(float a_, float c_) {
    const float s = 0x1p+40f;
    a = pack2(a_, a_); c = pack2(c_, c_);
    big = pack2(12582912.0f, 12582912.0f); nbig = pack2(-12582912.0f, -12582912.0f);
    none = pack2(-1.0f, -1.0f);
    c5 = pack2(0x1.5c7746p-10f * s, 0x1.5c7746p-10f * s); c4 = pack2(0x1.3cea8p-7f * s, 0x1.3cea8p-7f * s);
    c3 = pack2(0x1.c6b54ap-5f * s, 0x1.c6b54ap-5f * s); c2 = pack2(0x1.ebf9bcp-3f * s, 0x1.ebf9bcp-3f * s);
    c1 = pack2(0x1.62e42cp-1f * s, 0x1.62e42cp-1f * s); c0 = pack2(s, s);
  }
};
__device__ __forceinline__ unsigned long long weight_pair_sum(float z0, float z1, const WeightConsts2& k) {
  float y0, y1;
  unpack2(fma2(pack2(z0, z1), k.a, k.c), y0, y1);
  const unsigned long long y = pack2(fmaxf(y0, -42.0f), fmaxf(y1, -42.0f));
  const unsigned long long tmp = add2(y, k.big);
  const unsigned long long nf = add2(tmp, k.nbig);  // tmp - big
  const unsigned long long f = fma2(nf, k.none, y);  // y - nf, exact like the scalar subtraction
  unsigned long long p = fma2(k.c5, f, k.c4);
  p = fma2(p, f, k.c3);
  p = fma2(p, f, k.c2);
  p = fma2(p, f, k.c1);
  p = fma2(p, f, k.c0);
  float p0, p1, t0, t1;
  unpack2(p, p0, p1);
  unpack2(tmp, t0, t1);
  // the low mantissa bits of tmp hold n; shifted into the exponent field (the higher bits fall off the word)
  const uint32_t e0 = __float_as_uint(p0) + (__float_as_uint(t0) << 23);
  const uint32_t e1 = __float_as_uint(p1) + (__float_as_uint(t1) << 23);
  return __float2ull_rz(__uint_as_float(e0)) + __float2ull_rz(__uint_as_float(e1));
}
// Sum over the warp of per-lane sums below 2^46 (32 weights below 2^41 each): two 23-bit pieces, each summed
// by one warp-wide integer reduction.
__device__ __forceinline__ unsigned long long warp_sum_below_2p46(unsigned long long v) {
  const unsigned lo = (unsigned)v & 0x7fffffu, hi = (unsigned)(v >> 23);
  return (unsigned long long)__reduce_add_sync(FULL, lo) + ((unsigned long long)__reduce_add_sync(FULL, hi) << 23);
}

constexpr int G5_CHUNK = 1024;  // tokens per partial sum

// One warp: from the per-1024-token sums of a row's integer weights to the sampled token.  total = sum of
// the sums; theta = floor(R * total / 2^64) with R from Philox4x32-10(counter = (slot, b, 0, 0), key = seed);
// the pick is the first token whose inclusive prefix sum exceeds theta.  All lanes return the pick.
// theta = floor(R * total / 2^64), R the first two words of Philox4x32-10(counter = (slot, b, 0, 0), key = seed)
__device__ __forceinline__ unsigned long long sample_threshold(uint64_t seed, uint32_t b, uint32_t slot,
                                                               unsigned long long total) {
  uint32_t x[4];
  philox4x32_10(slot, b, 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), x);
  const unsigned long long R = (unsigned long long)x[0] | ((unsigned long long)x[1] << 32);
  return __umul64hi(R, total);
}

// One warp: the first token of rowp[0, V) whose inclusive prefix sum of weights exceeds theta (theta below the sum
// of all of them), from the per-1024-token sums csum.  All lanes return it.
template <typename T>
__device__ int locate_theta(const T* rowp, int V, float a, float c, const unsigned long long* csum, int nchunks,
                            unsigned long long theta, int lane) {
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
  int ans = t0 + G5_CHUNK / 32 - 1;
  if (lane == l) {
    unsigned long long run2 = inc - lsum;
    for (int j = 0; j < G5_CHUNK / 32; ++j) {
      const int tkn = t0 + j;
      run2 += tkn < V ? weight_of(load_elem(rowp, tkn), a, c) : 0ull;
      if (run2 > theta) { ans = tkn; break; }
    }
    ans = ans < V ? ans : V - 1;
  }
  return __shfl_sync(FULL, ans, l);
}

template <typename T>
__device__ int locate_pick(const T* rowp, int V, float a, float c, const unsigned long long* csum, int nchunks,
                           uint64_t seed, uint32_t b, uint32_t slot, int lane) {
  unsigned long long run = 0;
  for (int ch = lane; ch < nchunks; ch += 32) run += csum[ch];
  const unsigned long long total = warp_sum_u64(run);
  return locate_theta<T>(rowp, V, a, c, csum, nchunks, sample_threshold(seed, b, slot, total), lane);
}

// ---------------------------------------------------------------------------- sampling picks, ring-fed
// Every CTA owns whole rows and walks each of them twice through the bulk-copy ring: first for the row
// maximum, then (served by L2: a row is 0.3 MB and only one row per SM is in flight) for the integer weights,
// of which it stores one sum per 1024 tokens.  A second small kernel, one warp per row, turns the sums into
// the pick.  HBM traffic stays at one read of every logit; the weight arithmetic is what bounds this kernel.
constexpr int G5R_T = 512, G5R_STAGES = 3, G5R_STAGE_BYTES = 32768, G5R_CTAS = 2;

template <typename T>
struct RowTwiceProducer {  // thread 0: chunks of row r (pass 0), the same chunks again (pass 1), then row r+1
  static constexpr int kStageElems = G5R_STAGE_BYTES / (int)sizeof(T);
  int64_t row, row_end;
  int V, col, pass, stage, issued;
  uint64_t drop;  // L2 priority of the second pass: its lines will not be read again, so they go first and leave
                  // the room to the lines of first passes that still wait for their second (DRAM traffic 1.27 ->
                  // 1.06 x the logits; asking L2 to keep the first pass's lines as well changes nothing more)
  __device__ __forceinline__ void init(int64_t r0, int64_t r1, int V_) {
    row = r0; row_end = r1; V = V_; col = 0; pass = 0; stage = 0; issued = 0;
    drop = l2_policy_evict_first();
  }
  __device__ __forceinline__ void issue_one(const T* base, unsigned char* ring, uint64_t* full) {
    if (row >= row_end) return;
    const int l = V - col < kStageElems ? V - col : kStageElems;
    mbar_expect_tx(&full[stage], (uint32_t)(l * sizeof(T)));
    unsigned char* dst = ring + (size_t)stage * G5R_STAGE_BYTES;
    if (pass == 1) bulk_load_hint(dst, base + row * V + col, (uint32_t)(l * sizeof(T)), &full[stage], drop);
    else bulk_load(dst, base + row * V + col, (uint32_t)(l * sizeof(T)), &full[stage]);
    col += l;
    if (col == V) { col = 0; if (pass == 0) pass = 1; else { pass = 0; ++row; } }
    if (++stage == G5R_STAGES) stage = 0;
    ++issued;
  }
  __device__ __forceinline__ void drain(int consumed, uint64_t* full) {
    for (int i = consumed; i < issued; ++i) mbar_wait(&full[i % G5R_STAGES], (uint32_t)(i / G5R_STAGES) & 1u);
  }
};

template <typename T>
__global__ void __launch_bounds__(G5R_T, G5R_CTAS)
k_row_weights_ring(const T* __restrict__ logits, int64_t rows, int V, float temperature,
                   float* __restrict__ row_ac, unsigned long long* __restrict__ block_sum, int nblocks, int early) {
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ uint64_t full[G5R_STAGES];
  __shared__ float redf[G5R_T / 32];
  __shared__ int s_fail;
  constexpr int VEC = 16 / (int)sizeof(T);
  constexpr int STAGE_ELEMS = G5R_STAGE_BYTES / (int)sizeof(T);
  constexpr int BF = G5_CHUNK / VEC;  // fragments per 1024-token block
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t r0 = rows * blockIdx.x / gridDim.x, r1 = rows * (blockIdx.x + 1) / gridDim.x;
  if (!early) pdl_wait();  // stream order unless the caller opted into an early start (see k_row_argmax_ring)
  pdl_launch_dependents();
  if (r0 >= r1) {
    if (early && tid == 0) pdl_wait();
    return;
  }
  if (tid == 0) {
    for (int s = 0; s < G5R_STAGES; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_fail = 0;
  }
  __syncthreads();
  RowTwiceProducer<T> prod;
  if (tid == 0) {
    prod.init(r0, r1, V);
    for (int i = 0; i < G5R_STAGES - 1; ++i) prod.issue_one(logits, ring, full);
  }
  RingPos<G5R_STAGES> rp;
  rp.init();
  int consumed = 0;
  bool failed = false;
  const float inv_t = __fdiv_rn(1.0f, temperature);
  const float a = __fmul_rn(0x1.715476p+0f, inv_t);

  for (int64_t row = r0; row < r1 && !failed; ++row) {
    // ---- pass 1: the row maximum
    float m = -INFINITY;
    for (int c0 = 0; c0 < V; c0 += STAGE_ELEMS) {
      const int l = V - c0 < STAGE_ELEMS ? V - c0 : STAGE_ELEMS;
      if (*reinterpret_cast<volatile int*>(&s_fail)) { failed = true; break; }
      if (tid == 0) prod.issue_one(logits, ring, full);
      if (mbar_wait(&full[rp.stage], rp.parity)) {
        const uint4* stage = reinterpret_cast<const uint4*>(ring + (size_t)rp.stage * G5R_STAGE_BYTES);
        const int nfrag = l / VEC;
#pragma unroll 4
        for (int f = tid; f < nfrag; f += G5R_T) m = max_nan(m, frag_max(stage[f], (const T*)nullptr));
      } else {
        s_fail = 1;
      }
      __syncthreads();
      rp.next();
      ++consumed;
    }
    if (failed) break;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max_nan(m, __shfl_xor_sync(FULL, m, o));
    if (lane == 0) redf[warp] = m;
    __syncthreads();
    m = redf[0];
    for (int w = 1; w < G5R_T / 32; ++w) m = max_nan(m, redf[w]);
    const float c = -__fmul_rn(m, a);  // NaN / -inf for a row that holds a NaN / +inf: the pick kernel reports it
    if (tid == 0) { row_ac[row * 2] = a; row_ac[row * 2 + 1] = c; }
    WeightConsts2 wc;
    wc.init(a, c);
    // ---- pass 2: integer weights, one sum per 1024-token block (a warp owns a block)
    for (int c0 = 0; c0 < V; c0 += STAGE_ELEMS) {
      const int l = V - c0 < STAGE_ELEMS ? V - c0 : STAGE_ELEMS;
      if (*reinterpret_cast<volatile int*>(&s_fail)) { failed = true; break; }
      if (tid == 0) prod.issue_one(logits, ring, full);
      if (mbar_wait(&full[rp.stage], rp.parity)) {
        const uint4* stage = reinterpret_cast<const uint4*>(ring + (size_t)rp.stage * G5R_STAGE_BYTES);
        const int nfrag = l / VEC;
        const int nblk = (nfrag + BF - 1) / BF;
        for (int blk = warp; blk < nblk; blk += G5R_T / 32) {
          unsigned long long acc = 0;
          if ((blk + 1) * BF <= nfrag) {  // whole block: no bounds checks
#pragma unroll
            for (int q = 0; q < BF / 32; ++q) {
              Frag<T> x;
              x.unpack(stage[blk * BF + q * 32 + lane]);
#pragma unroll
              for (int j = 0; j < VEC; j += 2) acc += weight_pair_sum(x.x[j], x.x[j + 1], wc);
            }
          } else {
            for (int q = 0; q < BF / 32; ++q) {
              const int f = blk * BF + q * 32 + lane;
              if (f < nfrag) {
                Frag<T> x;
                x.unpack(stage[f]);
#pragma unroll
                for (int j = 0; j < VEC; j += 2) acc += weight_pair_sum(x.x[j], x.x[j + 1], wc);
              }
            }
          }
          static_assert((BF / 32) * VEC == 32, "a lane sums 32 weights per block");
          acc = warp_sum_below_2p46(acc);
          if (lane == 0) block_sum[row * nblocks + c0 / G5_CHUNK + blk] = acc;
        }
      } else {
        s_fail = 1;
      }
      __syncthreads();  // frees the stage; also separates redf's use in consecutive rows
      rp.next();
      ++consumed;
    }
  }
  __syncthreads();
  if (tid == 0 && *reinterpret_cast<volatile int*>(&s_fail)) {
    prod.drain(consumed > 0 ? consumed - 1 : 0, full);
    for (int64_t row = r0; row < r1; ++row) row_ac[row * 2] = -1.0f;  // a wait gave up: no scale is negative
  }
  if (early && tid == 0) pdl_wait();  // started early: do not complete before the kernel in front
}

// One warp per row: block sums -> pick.
template <typename T>
__global__ void __launch_bounds__(128)
k_row_pick(const T* __restrict__ logits, int64_t rows, int N, int V, uint64_t seed,
           const float* __restrict__ row_ac, const unsigned long long* __restrict__ block_sum, int nblocks,
           int32_t* __restrict__ pick) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  pdl_wait();
  pdl_launch_dependents();
  if (row >= rows) return;
  const float a = row_ac[row * 2], c = row_ac[row * 2 + 1];
  int ans;
  if (a < 0.f) ans = -2;                                   // the weights kernel gave up a wait on this row
  else if (!(c == c) || c == INFINITY || c == -INFINITY) ans = -1;  // row maximum NaN or +inf (c = -max * a)
  else ans = locate_pick<T>(logits + row * V, V, a, c, block_sum + row * nblocks, nblocks, seed, (uint32_t)(row / N),
                            (uint32_t)(row % N), lane);
  if (lane == 0) pick[row] = ans;
}

constexpr int G5_T = 512;

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
      for (int j = 0; j < VEC; ++j) m = max_nan(m, x[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max_nan(m, __shfl_xor_sync(FULL, m, o));
    __syncthreads();
    if (lane == 0) redf[warp] = m;
    __syncthreads();
    m = redf[0];
    for (int w = 1; w < G5_T / 32; ++w) m = max_nan(m, redf[w]);
    if (!(m == m) || m == INFINITY) {  // a NaN or +inf in the row: no pick, reported by the walk
      if (tid == 0) pick[row] = -1;
      __syncthreads();
      continue;
    }
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
      const int ans = locate_pick<T>(rowp, V, a, c, csum, nchunks, seed, (uint32_t)(row / N), (uint32_t)(row % N), lane);
      if (lane == 0) pick[row] = ans;
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------- the walk
// One CTA per sequence: gather the picks of its N slots, then warp 0 walks from the root.
__global__ void __launch_bounds__(128)
k_walk(ubt_tree tree, int mode, SpanPlan plan, const unsigned long long* __restrict__ part_key, int V,
       const int32_t* __restrict__ sampled_pick, int32_t* __restrict__ node_pick, ubt_verify_result out,
       int32_t* __restrict__ status, int shards, int64_t shard_stride) {
  __shared__ int s_pick[kMaxN], s_tok[kMaxN], s_par[kMaxN];
  __shared__ int s_bits;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, N = tree.N, L = tree.L;
  const int64_t o = (int64_t)b * N;
  if (tid == 0) s_bits = 0;
  pdl_wait();  // picks and tree come from the kernels before this one
  __syncthreads();
  for (int n = tid; n < N; n += blockDim.x) {
    int p, bits = 0;
    if (mode == UBT_VERIFY_GREEDY) {
      const int64_t row = o + n;
      // the keys of the row: one per segment of this GPU's row-argmax pass, or (shards > 0) one per rank of a
      // vocabulary-parallel group, rank r's keys `shard_stride` * r entries behind rank 0's
      int64_t nseg = shards, base = row, stride = shard_stride;
      if (shards == 0) {
        const int64_t c_first = (row * (int64_t)V) / plan.span;
        const int64_t c_last = ((row + 1) * (int64_t)V - 1) / plan.span;
        nseg = c_last - c_first + 1;
        base = row * plan.smax;
        stride = 1;
      }
      unsigned long long best = 0;
      for (int64_t j = 0; j < nseg; ++j) {
        const unsigned long long key = part_key[base + j * stride];
        best = key > best ? key : best;
      }
      p = best ? key_idx(best) : 0;  // a row without any comparable value falls back to token 0
      if (best == kKeyGaveUp) bits = kStatusWaitGaveUp;
      else if (best >= kKeyPlusInf) bits = kStatusNonFinite;  // +inf as the maximum, or the NaN marker
    } else {
      p = sampled_pick[o + n];
      // picks gathered from the ranks of a vocabulary-parallel group: the one rank that owns the slot's pick has a
      // token there, the others -1; no owner at all = no valid pick (the most severe marker is kept)
      int worst = p;
      for (int r = 1; r < shards; ++r) {
        const int q = sampled_pick[(int64_t)r * shard_stride + o + n];
        p = q > p ? q : p;
        worst = q < worst ? q : worst;
      }
      if (p < 0) p = worst;
      if (p < 0) { bits = p == -2 ? kStatusWaitGaveUp : kStatusNonFinite; p = 0; }
    }
    if (bits) atomicOr(&s_bits, bits);
    s_pick[n] = p;
    s_tok[n] = tree.token_ids[o + n];
    s_par[n] = tree.parents[o + n];
    if (node_pick) node_pick[o + n] = p;
  }
  __syncthreads();
  // Only now may a kernel behind this one become resident: the scratch (row keys / picks) has been read for the
  // last time, so an early-started pass of a following verify call cannot overwrite anything still needed here.
  pdl_launch_dependents();
  if (tid == 0 && status) status[b] = s_bits;
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
  return make_span_plan(rows, V, device_info().sm_count, 32768);
}

size_t verify_workspace_bytes(int64_t rows, int V, int mode) {
  if (mode == UBT_VERIFY_GREEDY) {
    const SpanPlan p = argmax_plan(rows, V);
    return align_up((size_t)rows * p.smax * sizeof(unsigned long long), 256);
  }
  const size_t nblocks = ((size_t)V + G5_CHUNK - 1) / G5_CHUNK;
  return align_up((size_t)rows * sizeof(int32_t), 256) + align_up((size_t)rows * 2 * sizeof(float), 256) +
         align_up((size_t)rows * nblocks * sizeof(unsigned long long), 256);
}

VerifyWorkspace carve_verify_workspace(void* ws, int64_t rows, int V, int mode) {
  VerifyWorkspace w{};
  if (mode == UBT_VERIFY_GREEDY) {
    w.plan = argmax_plan(rows, V);
    w.part_key = static_cast<unsigned long long*>(ws);
  } else {
    w.plan = SpanPlan{0, 0, 0};
    unsigned char* p = static_cast<unsigned char*>(ws);
    w.pick = reinterpret_cast<int32_t*>(p); p += align_up((size_t)rows * sizeof(int32_t), 256);
    w.row_ac = reinterpret_cast<float*>(p); p += align_up((size_t)rows * 2 * sizeof(float), 256);
    w.block_sum = reinterpret_cast<unsigned long long*>(p);
    w.nblocks = (V + G5_CHUNK - 1) / G5_CHUNK;
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

// Ring configuration of the greedy kernel: three stages, 256 threads, one CTA per SM.  Few large stages beat
// many small ones because every chunk pays a fixed latency.  The kernel is launched programmatically, so its
// CTAs should fit on an SM beside one CTA of the tree kernel that may still be resident in front of it: when
// the tree's tables leave no room for 3 x 64 KiB the stages shrink to 48 KiB.
constexpr int kArgmaxStages = 3, kArgmaxThreads = 256;
constexpr int kSmemPerSm = 228 * 1024, kSmemPerCtaReserved = 1024;

template <typename T, int STAGE_BYTES>
static cudaError_t launch_row_argmax_ring_t(const void* logits, int64_t rows, int V, const VerifyWorkspace& w,
                                            bool early, cudaStream_t st) {
  auto kern = k_row_argmax_ring<T, kArgmaxStages, STAGE_BYTES, kArgmaxThreads, 1>;
  constexpr int kBytes = kArgmaxStages * STAGE_BYTES;
  cudaError_t e = allow_max_dynamic_smem<k_row_argmax_ring<T, kArgmaxStages, STAGE_BYTES, kArgmaxThreads, 1>>();
  if (e != cudaSuccess) return e;
  // Always launched programmatically: the CTAs become resident behind the kernel in front.  Without `early`
  // they wait there until that kernel has completed before they read anything (plain stream order).
  return launch_kernel(kern, dim3(w.plan.grid), dim3(kArgmaxThreads), kBytes, st, true, static_cast<const T*>(logits),
                       rows * (int64_t)V, V, w.plan, w.part_key, early ? 1 : 0);
}

template <typename T>
static cudaError_t launch_row_argmax_ring_t(const void* logits, int64_t rows, int V, const VerifyWorkspace& w,
                                            size_t neighbour_smem, bool early, cudaStream_t st) {
  const bool roomy = kArgmaxStages * 65536 + neighbour_smem + 2 * kSmemPerCtaReserved <= (size_t)kSmemPerSm;
  return roomy ? launch_row_argmax_ring_t<T, 65536>(logits, rows, V, w, early, st)
               : launch_row_argmax_ring_t<T, 49152>(logits, rows, V, w, early, st);
}

cudaError_t launch_row_argmax(const void* logits, int dtype, int64_t rows, int V, const VerifyWorkspace& w,
                              size_t neighbour_smem, bool early, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  // rows that are whole 16-byte fragments go through the bulk-copy ring; other V use plain loads
  if (dtype == UBT_BF16 && V % 8 == 0) return launch_row_argmax_ring_t<__nv_bfloat16>(logits, rows, V, w, neighbour_smem, early, st);
  if (dtype == UBT_F32 && V % 4 == 0) return launch_row_argmax_ring_t<float>(logits, rows, V, w, neighbour_smem, early, st);
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

template <typename T>
static cudaError_t launch_row_sample_ring_t(const void* logits, int64_t rows, int N, int V, uint64_t seed,
                                            float temperature, int32_t* pick, const VerifyWorkspace& w,
                                            bool early, cudaStream_t st) {
  auto kern = k_row_weights_ring<T>;
  constexpr int kBytes = G5R_STAGES * G5R_STAGE_BYTES;
  cudaError_t e = allow_max_dynamic_smem<k_row_weights_ring<T>>();
  if (e != cudaSuccess) return e;
  int grid = device_info().sm_count * G5R_CTAS;
  if ((int64_t)grid > rows) grid = (int)rows;
  e = launch_kernel(kern, dim3(grid), dim3(G5R_T), kBytes, st, true, static_cast<const T*>(logits), rows, V,
                    temperature, w.row_ac, w.block_sum, w.nblocks, early ? 1 : 0);
  if (e != cudaSuccess) return e;
  const int warps = 4;
  return launch_kernel(k_row_pick<T>, dim3((unsigned)((rows + warps - 1) / warps)), dim3(warps * 32), 0, st, true,
                       static_cast<const T*>(logits), rows, N, V, seed, (const float*)w.row_ac,
                       (const unsigned long long*)w.block_sum, w.nblocks, pick);
}

cudaError_t launch_row_sample(const void* logits, int dtype, int B, int N, int V, uint64_t seed,
                              float temperature, int32_t* pick, const VerifyWorkspace& w, bool early,
                              cudaStream_t st) {
  const int64_t rows = (int64_t)B * N;
  if (rows == 0) return cudaSuccess;
  // rows that are whole 16-byte fragments go through the bulk-copy ring; other V use plain loads
  if (dtype == UBT_BF16 && V % 8 == 0)
    return launch_row_sample_ring_t<__nv_bfloat16>(logits, rows, N, V, seed, temperature, pick, w, early, st);
  if (dtype == UBT_F32 && V % 4 == 0)
    return launch_row_sample_ring_t<float>(logits, rows, N, V, seed, temperature, pick, w, early, st);
  if (dtype == UBT_BF16) {
    if (V % 8 == 0) return launch_row_sample_t<__nv_bfloat16, 8>(logits, rows, N, V, seed, temperature, pick, st);
    return launch_row_sample_t<__nv_bfloat16, 1>(logits, rows, N, V, seed, temperature, pick, st);
  }
  if (V % 4 == 0) return launch_row_sample_t<float, 4>(logits, rows, N, V, seed, temperature, pick, st);
  return launch_row_sample_t<float, 1>(logits, rows, N, V, seed, temperature, pick, st);
}

cudaError_t launch_walk(const ubt_tree& tree, int mode, const VerifyWorkspace& w, int V,
                        const int32_t* sampled_pick, int32_t* node_pick, const ubt_verify_result& out,
                        int32_t* status, cudaStream_t st, int pick_shards) {
  if (tree.B == 0) return cudaSuccess;
  return launch_kernel(k_walk, dim3(tree.B), dim3(128), 0, st, true, tree, mode, w.plan,
                       (const unsigned long long*)w.part_key, V, sampled_pick, node_pick, out, status,
                       mode == UBT_VERIFY_GREEDY ? 0 : pick_shards, (int64_t)tree.B * tree.N);
}

// Vocabulary-parallel greedy a4, first half: one key per row of this rank's slice -- the best key of the row's
// segments with its token moved by the slice's first column (the low word of a key is ~token; the marker keys of
// a non-finite or abandoned segment are kept as they are).
__global__ void __launch_bounds__(128)
k_row_keys_shard(SpanPlan plan, const unsigned long long* __restrict__ part_key, int64_t rows, int V, int v0,
                 unsigned long long* __restrict__ row_keys) {
  const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows) return;
  const int64_t c_first = (row * (int64_t)V) / plan.span;
  const int64_t c_last = ((row + 1) * (int64_t)V - 1) / plan.span;
  unsigned long long best = 0;
  for (int64_t j = 0; j <= c_last - c_first; ++j) {
    const unsigned long long key = part_key[row * plan.smax + j];
    best = key > best ? key : best;
  }
  if (best != 0ull && (best >> 32) <= (kKeyPlusInf >> 32))  // the key of a value (+inf included), not a marker
    best = (best & 0xffffffff00000000ull) | (unsigned long long)((uint32_t)best - (uint32_t)v0);
  row_keys[row] = best;
}

cudaError_t launch_row_keys_shard(const VerifyWorkspace& w, int64_t rows, int V, int v0, unsigned long long* row_keys,
                                  cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  k_row_keys_shard<<<(unsigned)((rows + 127) / 128), 128, 0, st>>>(w.plan, w.part_key, rows, V, v0, row_keys);
  return cudaGetLastError();
}

// Second half: the walk on the gathered keys ([shards, B*N], rank order).
cudaError_t launch_walk_keys(const ubt_tree& tree, const unsigned long long* gathered_keys, int shards,
                             int32_t* node_pick, const ubt_verify_result& out, int32_t* status, cudaStream_t st) {
  if (tree.B == 0) return cudaSuccess;
  return launch_kernel(k_walk, dim3(tree.B), dim3(128), 0, st, true, tree, (int)UBT_VERIFY_GREEDY, SpanPlan{},
                       gathered_keys, 1, (const int32_t*)nullptr, node_pick, out, status, shards,
                       (int64_t)tree.B * tree.N);
}

// ------------------------------------------------------- sampling a4 with the vocabulary split over ranks
// The integer weights make the split exact: with the row maximum taken over ALL ranks' slices (from the gathered
// keys of the greedy pass), every rank computes the weights of its own columns with the same (a, c) as one GPU
// would, the row total is the sum of the ranks' totals, theta follows from it, and the rank whose share of the
// running sum holds theta finds the token in its slice.
//
// First half: per row the global maximum from the gathered keys, (a, c), the per-1024-token sums of this slice's
// weights (kept in the workspace for the second half) and their total.
template <typename T, int VEC>
__global__ void __launch_bounds__(G5_T, 2)
k_row_totals_shard(const T* __restrict__ logits, int64_t rows, int Vs, const unsigned long long* __restrict__ gathered_keys,
                   int shards, float temperature, float* __restrict__ row_ac, unsigned long long* __restrict__ block_sum,
                   int nblocks, unsigned long long* __restrict__ totals) {
  __shared__ unsigned long long wsum[G5_T / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int CF = G5_CHUNK / VEC;  // fragments per chunk
  const float inv_t = __fdiv_rn(1.0f, temperature);
  const float a = __fmul_rn(0x1.715476p+0f, inv_t);
  for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
    unsigned long long best = 0;
    for (int r = 0; r < shards; ++r) {
      const unsigned long long key = gathered_keys[(int64_t)r * rows + row];
      best = key > best ? key : best;
    }
    // a marker key (a NaN or +inf somewhere in the row, an abandoned wait) or no key at all: no pick for this row
    float a_row = a, c = __uint_as_float(0x7fc00000u);
    if (best == kKeyGaveUp) a_row = -1.0f;
    else if (best != 0ull && best < kKeyPlusInf) c = -__fmul_rn(key_val(best), a);
    const bool live = a_row >= 0.f && c == c && c != INFINITY && c != -INFINITY;
    if (tid == 0) { row_ac[row * 2] = a_row; row_ac[row * 2 + 1] = c; }
    unsigned long long wtot = 0;
    if (live) {
      const T* rowp = logits + row * Vs;
      const int nfrag = Vs / VEC;  // Vs % VEC == 0 on the vector path; VEC == 1 otherwise
      for (int ch = warp; ch < nblocks; ch += G5_T / 32) {
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
        if (lane == 0) block_sum[row * nblocks + ch] = acc;
        wtot += acc;
      }
    }
    if (lane == 0) wsum[warp] = wtot;
    __syncthreads();
    if (tid == 0) {
      unsigned long long t = 0;
      for (int w = 0; w < G5_T / 32; ++w) t += wsum[w];
      totals[row] = t;
    }
    __syncthreads();
  }
}

// Second half, one warp per row: theta from the sum of the ranks' totals; the rank whose share [before, before +
// own total) holds theta writes the token (counted in the whole vocabulary), every other rank -1.  A row without a
// valid maximum gets -1 (-2 after an abandoned wait) from every rank.
template <typename T>
__global__ void __launch_bounds__(128)
k_row_pick_shard(const T* __restrict__ logits, int64_t rows, int N, int Vs, int v0, int rank, int shards,
                 const unsigned long long* __restrict__ gathered_totals, uint64_t seed, const float* __restrict__ row_ac,
                 const unsigned long long* __restrict__ block_sum, int nblocks, int32_t* __restrict__ pick) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float a = row_ac[row * 2], c = row_ac[row * 2 + 1];
  int ans = -1;
  if (a < 0.f) {
    ans = -2;
  } else if (c == c && c != INFINITY && c != -INFINITY) {
    unsigned long long total = 0, before = 0;
    for (int r = 0; r < shards; ++r) {
      const unsigned long long t = gathered_totals[(int64_t)r * rows + row];
      if (r < rank) before += t;
      total += t;
    }
    const unsigned long long mine = gathered_totals[(int64_t)rank * rows + row];
    const unsigned long long theta = sample_threshold(seed, (uint32_t)(row / N), (uint32_t)(row % N), total);
    if (theta >= before && theta - before < mine)
      ans = v0 + locate_theta<T>(logits + row * Vs, Vs, a, c, block_sum + row * nblocks, nblocks, theta - before, lane);
  }
  if (lane == 0) pick[row] = ans;
}

cudaError_t launch_row_totals_shard(const void* logits, int dtype, int64_t rows, int Vs,
                                    const unsigned long long* gathered_keys, int shards, float temperature,
                                    const VerifyWorkspace& w, unsigned long long* totals, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  const int grid = (int)(rows < 4096 ? rows : 4096);
  if (dtype == UBT_BF16) {
    if (Vs % 8 == 0)
      k_row_totals_shard<__nv_bfloat16, 8><<<grid, G5_T, 0, st>>>(static_cast<const __nv_bfloat16*>(logits), rows, Vs, gathered_keys,
                                                                   shards, temperature, w.row_ac, w.block_sum, w.nblocks, totals);
    else
      k_row_totals_shard<__nv_bfloat16, 1><<<grid, G5_T, 0, st>>>(static_cast<const __nv_bfloat16*>(logits), rows, Vs, gathered_keys,
                                                                   shards, temperature, w.row_ac, w.block_sum, w.nblocks, totals);
  } else if (Vs % 4 == 0) {
    k_row_totals_shard<float, 4><<<grid, G5_T, 0, st>>>(static_cast<const float*>(logits), rows, Vs, gathered_keys, shards,
                                                        temperature, w.row_ac, w.block_sum, w.nblocks, totals);
  } else {
    k_row_totals_shard<float, 1><<<grid, G5_T, 0, st>>>(static_cast<const float*>(logits), rows, Vs, gathered_keys, shards,
                                                        temperature, w.row_ac, w.block_sum, w.nblocks, totals);
  }
  return cudaGetLastError();
}

cudaError_t launch_row_pick_shard(const void* logits, int dtype, int64_t rows, int N, int Vs, int v0, int rank, int shards,
                                  const unsigned long long* gathered_totals, uint64_t seed, const VerifyWorkspace& w,
                                  int32_t* pick, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  const unsigned grid = (unsigned)((rows + 3) / 4);
  if (dtype == UBT_BF16)
    k_row_pick_shard<__nv_bfloat16><<<grid, 128, 0, st>>>(static_cast<const __nv_bfloat16*>(logits), rows, N, Vs, v0, rank, shards,
                                                          gathered_totals, seed, w.row_ac, w.block_sum, w.nblocks, pick);
  else
    k_row_pick_shard<float><<<grid, 128, 0, st>>>(static_cast<const float*>(logits), rows, N, Vs, v0, rank, shards,
                                                  gathered_totals, seed, w.row_ac, w.block_sum, w.nblocks, pick);
  return cudaGetLastError();
}

// Number of bounded waits that gave up in this file's kernels (0 in a healthy run).
cudaError_t ring_timeouts_verify(unsigned int* out) { return cudaMemcpyFromSymbol(out, g_ring_timeouts, sizeof *out); }

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
