// Steps a2, a3, a3b: candidate-pair log-probabilities, budgeted tree expansion, tree-attention inputs.
//
// One CTA per sequence.  The pair table t[i][ra][.] = log q^bi (eq. 5 + eq. 9) lives in shared memory,
// every row sorted best first, next to the permutation that sorted it.  Every pair log-probability is <= 0 and
// zeta <= 0, so scores never increase from a node to its children or to its later siblings; Algorithm 1 (Top_W per
// depth, eq. 11, then the global Top_B, eq. 12) is evaluated in two equivalent ways that both rest on that:
//   * threshold rounds (the whole table resident): the nodes that reach a threshold form a set closed under
//     "parent" and "earlier sibling" that is enumerated in parallel, wave by wave; the threshold falls from round
//     to round until the set covers the budget, and the budget's best nodes of the last round are chosen under the
//     total order (score desc, depth asc, token asc, rank path asc).  See expand_rounds_warp / expand_rounds_cta.
//   * best-first search by one warp (pair table too large for shared memory, rows prepared on demand; also the
//     fallback when masses of exactly tied scores outgrow the rounds' node arrays): the frontier holds, per
//     expanded node, its best not-yet-taken child; a pop takes the best entry, replaces it by its next sibling
//     and adds its own first child, so pops come out in the global order; a node popped when its depth already
//     holds W nodes is outside Top_W(E_d) and is dropped with its later siblings.  See expand_tree.
// Everything around the search -- merging the top-k partials, eq. 5 / eq. 9 and the row sorts, slot assignment,
// masks -- is spread over the CTA's 16 warps.
#include "ubt_internal.h"

namespace ubt {

constexpr int G2_T = 512;

struct TreeSmem {
  // Pair log-probabilities, one row per (position, predecessor rank), each row sorted descending, next to the
  // permutation that sorted it (ord[row][j] = candidate rank of the j-th best successor).  Whole table [L,k,k]
  // when it fits; otherwise a cache of the rows the search touches ([N,k]: a pop opens at most one new row),
  // filled on demand and found through `rowmap`.
  Span<float> t;
  Span<unsigned char> ord;
  Span<short> rowmap;       // lazy mode: [L*k + 1] cache slot of row (position * k + predecessor rank), -1 = not yet
  Span<float> la;           // [L]    eq. 5 weight of the selector score per position
  Span<float> pre;          // lazy mode: [N+1][k] raw selector scores of the row each frontier record will open
  Span<float> lp;           // [L,k]
  Span<int> tok;            // [L,k]
  Span<float> al;           // [L]    eq. 5 weight of the base log-probability per position
  Span<uint4> ent;          // [N+1]  frontier records of the expansion
  Span<short> nd_parent;    // accepted nodes in pop order, <= N-1; -1 = child of the root
  Span<unsigned char> nd_depth;
  Span<unsigned char> nd_rank;
  Span<float> nd_score;
  Span<short> nd_slot;
  Span<unsigned long long> nd_pk;  // [N,2] rank path packed big-endian (hi, lo): lexicographic = numeric
  Span<int> kk;             // per-depth sort keys (fallback slot assignment)
  Span<int> depth_cnt;      // [L+2]
  Span<int> depth_off;      // [L+2]
  Span<int> x_fill;         // [L+2] fill counters of the grouping by depth
  Span<uint32_t> maskrow;   // [N, mask_words]
  Span<int> scalars;        // [0] accepted count, [1]-[3] scratch of the expansion, [4] status bits of the sequence
  // Nodes enumerated by the parallel expansion (resident table only; see expand_rounds): node 0 is the root.
  int xcap;                 // capacity (lazy mode: 0, or that of the depth-by-depth expansion)
  Span<short> x_parent;     // [xcap] enumerated parent, -1 for the root
  Span<unsigned char> x_depth, x_rank, x_next, x_bak;  // [xcap] depth, candidate rank, next child to enumerate (+ its backup)
  Span<float> x_score;      // [xcap]
  Span<uint32_t> x_key;     // [xcap] ordering key of the node's best child not yet enumerated, 0 = none
  Span<short> x_aux;        // [xcap] per-round scratch
  Span<unsigned long long> x_key64;  // [xcap] ordering keys of the final choice
  Span<int> x_wsum;         // [32] warp totals of the block scans
  Span<unsigned long long> dw_row;  // [warps, max(32, k rounded up to 4)] ordering keys of the rows a warp is ranking
  Span<uint32_t> dw_ckey;           // depth-by-depth expansion: score keys of a depth's candidates, packed
};

// Rows of the pair table are computed on demand when the whole table would not fit.
__host__ __device__ inline bool tree_lazy(int L, int k) { return (size_t)L * k * k * 5 > kTreeTableBytes; }
// Nodes the parallel expansion may enumerate before it picks the N - 1 best (root included).
__host__ __device__ inline int expand_capacity(int N) { return 4 * N < 128 ? 128 : (4 * N > 1024 ? 1024 : 4 * N); }
// A small finite width: eq. 11 runs depth by depth (expand_depthwise) on rows normalised on demand, whether or not
// the pair table would fit -- the search opens W rows per depth, and preparing just those is cheaper than the
// whole table.  The node arrays then hold the root and W nodes per depth, followed by a scratch area for the
// W * min(W, k) candidates of one depth.
constexpr int kDepthwiseMaxW = 16;
__host__ __device__ inline int depthwise_capacity(int L, int k, int N, int W) {
  if (W <= 0 || W >= N - 1 || W > kDepthwiseMaxW) return 0;
  return 1 + W * L + W * (W < k ? W : k);
}

// Byte offsets of the arrays above inside the CTA's dynamic shared memory.  They depend on L, k, N only, so
// the host computes them once per launch and passes them as a kernel argument: the kernel then forms every
// address from a constant-bank operand instead of keeping (or re-deriving) thirty pointers in registers.
struct TreeLayout {
  uint32_t t, ord, rowmap, la, pre, lp, tok, al, ent, nd_parent, nd_depth, nd_rank, nd_score, nd_slot, nd_pk, kk,
      depth_cnt, depth_off, x_fill, maskrow, scalars, x_parent, x_depth, x_rank, x_next, x_bak, x_score, x_key, x_aux,
      x_wsum, x_key64, dw_row, dw_ckey;
  uint32_t total;
  int xcap;
  int lazy;
};

inline TreeLayout tree_layout(int L, int k, int N, int W = 0) {
  TreeLayout o{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off = (off + bytes + 15) / 16 * 16;
    return (uint32_t)at;
  };
  const int mw = (N + 31) / 32;
  const bool lazy = tree_lazy(L, k) || depthwise_capacity(L, k, N, W) > 0;  // rows on demand
  const long long lkk = lazy ? (long long)N * k : (long long)L * k * k, lk = (long long)L * k;
  o.t = take(sizeof(float) * lkk); o.ord = take((size_t)lkk);
  o.rowmap = take(lazy ? sizeof(short) * (lk + 1) : 0); o.la = take(sizeof(float) * L);
  o.pre = take(lazy ? sizeof(float) * (size_t)(N + 1) * k : 0);
  o.lp = take(sizeof(float) * lk); o.tok = take(sizeof(int) * lk);
  o.al = take(sizeof(float) * L); o.ent = take(sizeof(uint4) * (N + 1));
  o.nd_parent = take(sizeof(short) * N); o.nd_depth = take(N); o.nd_rank = take(N);
  o.nd_score = take(sizeof(float) * N); o.nd_slot = take(sizeof(short) * N);
  o.nd_pk = take(sizeof(unsigned long long) * 2 * N); o.kk = take(sizeof(int) * N);
  o.depth_cnt = take(sizeof(int) * (L + 2)); o.depth_off = take(sizeof(int) * (L + 2));
  o.x_fill = take(sizeof(int) * (L + 2));
  o.maskrow = take(sizeof(uint32_t) * N * mw); o.scalars = take(sizeof(int) * 8);
  const int xcap = lazy ? depthwise_capacity(L, k, N, W) : expand_capacity(N);
  o.xcap = xcap;
  o.lazy = lazy ? 1 : 0;
  o.x_parent = take(sizeof(short) * xcap); o.x_depth = take(xcap); o.x_rank = take(xcap); o.x_next = take(xcap);
  o.x_bak = take(xcap); o.x_score = take(sizeof(float) * xcap); o.x_key = take(sizeof(uint32_t) * xcap);
  o.x_aux = take(sizeof(short) * xcap); o.x_wsum = take(sizeof(int) * 32);
  o.x_key64 = take(sizeof(unsigned long long) * xcap);
  o.dw_row = take(sizeof(unsigned long long) * (G2_T / 32) * (((k + 3) & ~3) < 32 ? 32 : ((k + 3) & ~3)));
  o.dw_ckey = take(sizeof(uint32_t) * kDepthwiseMaxW * kDepthwiseMaxW);
  o.total = (uint32_t)off;
  return o;
}

__device__ __forceinline__ void tree_bind(TreeSmem* s, unsigned char* base, const TreeLayout& o, int L, int k, int N) {
  const int mw = (N + 31) / 32, xcap = o.xcap;
  const bool lazy = o.lazy != 0;
  const long long lkk = lazy ? (long long)N * k : (long long)L * k * k, lk = (long long)L * k;
  s->xcap = xcap;
  s->x_parent = Span<short>((short*)(base + o.x_parent), xcap, 121);
  s->x_depth = Span<unsigned char>(base + o.x_depth, xcap, 122);
  s->x_rank = Span<unsigned char>(base + o.x_rank, xcap, 123);
  s->x_next = Span<unsigned char>(base + o.x_next, xcap, 124);
  s->x_bak = Span<unsigned char>(base + o.x_bak, xcap, 125);
  s->x_score = Span<float>((float*)(base + o.x_score), xcap, 126);
  s->x_key = Span<uint32_t>((uint32_t*)(base + o.x_key), xcap, 127);
  s->x_aux = Span<short>((short*)(base + o.x_aux), xcap, 128);
  s->x_wsum = Span<int>((int*)(base + o.x_wsum), 32, 129);
  s->x_key64 = Span<unsigned long long>((unsigned long long*)(base + o.x_key64), xcap, 130);
  s->dw_row = Span<unsigned long long>((unsigned long long*)(base + o.dw_row), (long long)(G2_T / 32) * (((k + 3) & ~3) < 32 ? 32 : ((k + 3) & ~3)), 131);
  s->dw_ckey = Span<uint32_t>((uint32_t*)(base + o.dw_ckey), kDepthwiseMaxW * kDepthwiseMaxW, 132);
  s->t = Span<float>((float*)(base + o.t), lkk, 101);
  s->ord = Span<unsigned char>(base + o.ord, lkk, 102);
  s->rowmap = Span<short>((short*)(base + o.rowmap), lazy ? lk + 1 : 0, 107);
  s->la = Span<float>((float*)(base + o.la), L, 108);
  s->pre = Span<float>((float*)(base + o.pre), lazy ? (long long)(N + 1) * k : 0, 120);
  s->lp = Span<float>((float*)(base + o.lp), lk, 103);
  s->tok = Span<int>((int*)(base + o.tok), lk, 104);
  s->al = Span<float>((float*)(base + o.al), L, 105);
  s->ent = Span<uint4>((uint4*)(base + o.ent), N + 1, 106);
  s->nd_parent = Span<short>((short*)(base + o.nd_parent), N, 109);
  s->nd_depth = Span<unsigned char>(base + o.nd_depth, N, 110);
  s->nd_rank = Span<unsigned char>(base + o.nd_rank, N, 111);
  s->nd_score = Span<float>((float*)(base + o.nd_score), N, 112);
  s->nd_slot = Span<short>((short*)(base + o.nd_slot), N, 113);
  s->nd_pk = Span<unsigned long long>((unsigned long long*)(base + o.nd_pk), 2LL * N, 114);
  s->kk = Span<int>((int*)(base + o.kk), N, 115);
  s->depth_cnt = Span<int>((int*)(base + o.depth_cnt), L + 2, 116);
  s->depth_off = Span<int>((int*)(base + o.depth_off), L + 2, 117);
  s->x_fill = Span<int>((int*)(base + o.x_fill), L + 2, 131);
  s->maskrow = Span<uint32_t>((uint32_t*)(base + o.maskrow), (long long)N * mw, 118);
  s->scalars = Span<int>((int*)(base + o.scalars), 8, 119);
}

size_t tree_smem_bytes(int L, int k, int N) { return tree_layout(L, k, N).total; }

// A frontier entry is one 16-byte record in shared memory (entry i belongs to lane i & 31, slot i >> 5); only
// its ordering key is mirrored in a register of the owner lane, so that finding the best entry is a register
// scan and one warp-wide maximum.  The record holds all a pop needs:
//   x: parent node (8 bits, 255 = the root) | sibling position j (6) | depth - 1 (6) | own candidate rank (6)
//   y: index of its value in the sorted pair table (15 bits) | index of its first child's row (15 bits)
//   z: score of its parent (float bits)     w: ordering key of its own score, 0 = dead
__device__ __forceinline__ uint32_t pack_lo(int p, int j, int d, int r) {
  return (uint32_t)p | ((uint32_t)j << 8) | ((uint32_t)(d - 1) << 14) | ((uint32_t)r << 20);
}

// Lazy mode.  The raw selector scores of a row are fetched ahead of time: when a record enters the frontier, the
// row its node would open (position = its depth, predecessor = its rank) is copied asynchronously from global
// memory into the record's prefetch slot, so the copy's latency has passed long before the node is popped.
struct RowSource {
  const float* bigram;         // this sequence's [L-1,k,k] selector scores
  const float* anchor_bigram;  // this sequence's [k] or nullptr
};
__device__ __forceinline__ void cp_async_f32(float* smem_dst, const float* gmem_src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
               : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// row q = i * k + ra into prefetch slot e (k <= 64: a lane copies elements lane and lane + 32)
__device__ __forceinline__ void prefetch_row(TreeSmem& s, const RowSource& src, int q, int e, int k, int L, int lane) {
  const int i = q / k, ra = q - i * k;
  if (i >= L) return;
  const float* row = i == 0 ? src.anchor_bigram : src.bigram + ((size_t)(i - 1) * k + ra) * k;
  float* dst = s.pre.ptr((long long)e * k, k);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int rb = lane + 32 * h;
    if (rb < k) {
      if (row) cp_async_f32(dst + rb, row + rb);
      else dst[rb] = 0.f;  // no anchor scores: zeros
    }
  }
}
// One warp ranks the k <= 64 entries of a row (two per lane: lane and lane + 32) under (value desc, token asc): the
// 32-bit value keys meet in the warp's scratch and every lane counts the keys in front of its two entries -- k
// independent shared-memory loads and 2 k compares, no warp-wide reductions, no extraction rounds.  Equal values
// (rare) would give two entries the same rank: every entry marks the place of its rank with its index, an entry
// that finds another index there was tied, and the warp then counts again with the full (value key, ~token) keys,
// which are distinct because the candidates of a position are distinct tokens.  k64[h] receives the full keys.
__device__ __forceinline__ void rank_row_warp(TreeSmem& s, const float (&v)[2], const uint32_t (&ntok)[2], int k, int lane,
                                              unsigned long long (&k64)[2], int& r0, int& r1) {
  const int kpad = (k + 3) & ~3;
  unsigned long long* rowkeys = s.dw_row.ptr((long long)(threadIdx.x >> 5) * kpad, kpad);
  uint32_t* key32 = reinterpret_cast<uint32_t*>(rowkeys);      // [kpad] value keys (0 = none), then [kpad] marks
  uint32_t kv[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int rb = lane + 32 * h;
    kv[h] = f2key(v[h]);
    kv[h] = kv[h] == 0u ? 1u : kv[h];
    k64[h] = ((unsigned long long)kv[h] << 32) | ntok[h];
    if (rb < kpad) key32[rb] = rb < k ? kv[h] : 0u;
  }
  __syncwarp();
  // four keys per load and eight independent counters: a single warp issues a dependent instruction only every
  // few cycles, so the loop is a matter of keeping independent work in flight
  const uint4* key128 = reinterpret_cast<const uint4*>(key32);
  int a0 = 0, a1 = 0, a2 = 0, a3 = 0, b0 = 0, b1 = 0, b2 = 0, b3 = 0;
#pragma unroll 4
  for (int j = 0; j < kpad / 4; ++j) {
    const uint4 q = key128[j];
    a0 += q.x > kv[0]; a1 += q.y > kv[0]; a2 += q.z > kv[0]; a3 += q.w > kv[0];
    b0 += q.x > kv[1]; b1 += q.y > kv[1]; b2 += q.z > kv[1]; b3 += q.w > kv[1];
  }
  r0 = (a0 + a1) + (a2 + a3);
  r1 = (b0 + b1) + (b2 + b3);
  // a place per rank: ties collide
  if (lane < k) key32[kpad + r0] = (uint32_t)lane;
  if (lane + 32 < k) key32[kpad + r1] = (uint32_t)(lane + 32);
  __syncwarp();
  const bool clash = (lane < k && key32[kpad + r0] != (uint32_t)lane) || (lane + 32 < k && key32[kpad + r1] != (uint32_t)(lane + 32));
  if (__any_sync(FULL, clash)) {  // equal values in the row: rank again on (value key, ~token)
    __syncwarp();
#pragma unroll
    for (int h = 0; h < 2; ++h)
      if (lane + 32 * h < k) rowkeys[lane + 32 * h] = k64[h];
    __syncwarp();
    r0 = 0; r1 = 0;
    for (int j = 0; j < k; ++j) {
      const unsigned long long kj = rowkeys[j];
      r0 += kj > k64[0];
      r1 += kj > k64[1];
    }
  }
  __syncwarp();  // the scratch may be overwritten by the warp's next row
}

// One warp: eq. 5 and eq. 9 for row q from the raw scores in prefetch slot e, then its `m` best successors under
// (t desc, token asc) into cache slot `slot` (the search never looks further down a row: at most W, or the whole
// budget, of its entries can be accepted, plus one that is dropped).  The candidates of a position are distinct
// tokens, so (value key, ~token) orders a row strictly.
__device__ __forceinline__ void lazy_row(TreeSmem& s, int q, int e, int slot, int k, int m, int lane) {
  const int i = q / k;
  const float al = s.al[i], la = s.la[i];
  cp_async_wait_all();
  __syncwarp();
  float v[2];
  uint32_t ntok[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int rb = lane + 32 * h;
    v[h] = -INFINITY;
    ntok[h] = 0u;
    if (rb < k) {
      v[h] = fmaf(al, s.lp[i * k + rb], la * s.pre[(long long)e * k + rb]);
      ntok[h] = ~(uint32_t)s.tok[i * k + rb];
    }
  }
  float mx = fmaxf(v[0], v[1]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
  float sum = (lane < k ? expf(v[0] - mx) : 0.f) + (lane + 32 < k ? expf(v[1] - mx) : 0.f);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
  const float lse = mx + logf(sum);
  v[0] -= lse; v[1] -= lse;
  unsigned long long k64[2];
  int r0, r1;
  rank_row_warp(s, v, ntok, k, lane, k64, r0, r1);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int rb = lane + 32 * h, r = h == 0 ? r0 : r1;
    if (rb < k && r < m) {
      s.t[(long long)slot * k + r] = v[h];
      s.ord[(long long)slot * k + r] = (unsigned char)rb;
    }
  }
  __syncwarp();
}

// Best-first expansion by one warp; returns the number of accepted nodes (all lanes agree).
// Writes the accepted nodes in pop order: nd_parent, nd_depth, nd_rank, nd_score.
// A record's y word holds the index of its value in the table (15 bits) and the row number q = depth * k + rank
// of its node's children (13 bits); with the whole table resident that row starts at q * k, in lazy mode at
// rowmap[q] * k, computed when the node is popped for the first time.
template <int SLOTS, bool LAZY>
__device__ __forceinline__ int expand_tree(TreeSmem& s, const RowSource& src, int L, int k, int budget, int W, float zeta, int lane) {
  uint32_t fk[SLOTS];
#pragma unroll
  for (int q = 0; q < SLOTS; ++q) fk[q] = 0u;
  int f_cnt = 0, n_acc = 0, n_rows = 0;
  // entries of a row the search can reach (see lazy_row); with the whole table resident rows are fully sorted
  const int row_len = LAZY ? min(k, (W > 0 ? W : budget) + 1) : k;
  if (budget > 0) {
    if (LAZY) {
      prefetch_row(s, src, 0, 0, k, L, lane);
      lazy_row(s, 0, 0, 0, k, row_len, lane);
      n_rows = 1;
    }
    const int r0 = s.ord[0];
    const uint32_t key0 = f2key(s.t[0] + zeta);
    if (lane == 0) fk[0] = key0;
    s.ent[0] = make_uint4(pack_lo(255, 0, 1, r0), (uint32_t)(k + r0) << 15, __float_as_uint(0.f), key0);
    if (LAZY && L > 1) prefetch_row(s, src, k + r0, 0, k, L, lane);  // the row this first record would open
    f_cnt = 1;
  }
  __syncwarp();
  while (n_acc < budget) {
    uint32_t bk = fk[0];
    int bs = 0;
    bool dup = false;
#pragma unroll
    for (int q = 1; q < SLOTS; ++q) {
      dup = fk[q] > bk ? false : (dup || (fk[q] == bk && bk != 0u));
      bs = fk[q] > bk ? q : bs;
      bk = fk[q] > bk ? fk[q] : bk;
    }
    const uint32_t maxk = __reduce_max_sync(FULL, bk);
    if (maxk == 0u) break;  // frontier exhausted
    // who holds it: lane | slot << 5 | (two equal keys in that lane) << 8; minimum and maximum over the
    // holders agree iff there is one holder
    const uint32_t code = (uint32_t)lane | ((uint32_t)bs << 5) | (dup ? 256u : 0u);
    const uint32_t cmin = __reduce_min_sync(FULL, bk == maxk ? code : 0xffffffffu);
    const uint32_t cmax = __reduce_max_sync(FULL, bk == maxk ? code : 0u);
    int wl = (int)(cmin & 31u), ws = (int)((cmin >> 5) & 7u);
    if (cmin != cmax || (cmin & 256u)) {
      // Exact score ties (rare): depth asc, token asc, then rank path lexicographic, decided redundantly
      // on all lanes from the records in shared memory.
      int best = -1, bd = 0, bt = 0;
      uint32_t best_lo = 0;
      for (int i = 0; i < f_cnt; ++i) {
        const uint4 e = s.ent[i];
        if (e.w != maxk) continue;
        const uint32_t el = e.x;
        const int d = (int)((el >> 14) & 63u) + 1, r = (int)((el >> 20) & 63u);
        const int tkn = s.tok[(d - 1) * k + r];
        bool better;
        if (best < 0) better = true;
        else if (d != bd) better = d < bd;
        else if (tkn != bt) better = tkn < bt;
        else {  // same depth and token: the shallowest level where the two prefixes differ decides
          int pa = (int)(el & 255u), pb = (int)(best_lo & 255u), ra = 0, rb = 0;
          pa = pa == 255 ? -1 : pa; pb = pb == 255 ? -1 : pb;
          while (pa != pb) {
            ra = s.nd_rank[pa]; rb = s.nd_rank[pb];
            pa = s.nd_parent[pa]; pb = s.nd_parent[pb];
          }
          better = ra < rb;
        }
        if (better) { best = i; bd = d; bt = tkn; best_lo = el; }
      }
      wl = best & 31;
      ws = best >> 5;
    }
    const int e_idx = ws * 32 + wl;
    const uint4 ent = s.ent[e_idx];
    const uint32_t lo = ent.x, hi = ent.y;
    const float ps = __uint_as_float(ent.z);
    const int p = (int)(lo & 255u), j = (int)((lo >> 8) & 63u), d = (int)((lo >> 14) & 63u) + 1;
    const int r = (int)((lo >> 20) & 63u), at = (int)(hi & 0x7fffu), qrow = (int)((hi >> 15) & 0x1fffu);
    const float score = key2f(maxk);
    if (W > 0) {
      const int dc = s.depth_cnt[d];
      if (dc >= W) {  // outside Top_W(E_d); so are its later siblings
#pragma unroll
        for (int q = 0; q < SLOTS; ++q) fk[q] = (lane == wl && q == ws) ? 0u : fk[q];
        s.ent[e_idx] = make_uint4(0u, 0u, 0u, 0u);
        __syncwarp();
        continue;
      }
      s.depth_cnt[d] = dc + 1;
    }
    // one round of independent loads: next sibling and first child
    const bool has_sib = j + 1 < row_len, has_child = d < L;
    int cb = qrow * k;
    if (LAZY && has_child) {  // the row of this node's children: open it on first use
      int slot = s.rowmap[qrow];
      if (slot < 0) {
        slot = n_rows++;
        lazy_row(s, qrow, e_idx, slot, k, row_len, lane);
        if (lane == 0) s.rowmap[qrow] = (short)slot;
        __syncwarp();
      }
      cb = slot * k;
    }
    const int i_sib = has_sib ? at + 1 : 0, i_child = has_child ? cb : 0;
    const float t_sib = s.t[i_sib], t_child = s.t[i_child];
    const int r_sib = s.ord[i_sib], r_child = s.ord[i_child];
    // Every store below is executed by all lanes with the same address and value: a divergent single-lane
    // block costs more than the whole rest of the pop.
    const int n = n_acc++;
    s.nd_parent[n] = (short)(p == 255 ? -1 : p);
    s.nd_depth[n] = (unsigned char)d;
    s.nd_rank[n] = (unsigned char)r;
    s.nd_score[n] = score;
    const uint32_t k_sib = has_sib ? f2key(ps + t_sib + zeta) : 0u;
    const uint32_t k_child = has_child ? f2key(score + t_child + zeta) : 0u;
    const int cl = f_cnt & 31, cs = f_cnt >> 5;
    s.ent[e_idx] = make_uint4(pack_lo(p, j + 1, d, r_sib), (uint32_t)i_sib | ((uint32_t)(d * k + r_sib) << 15),
                              ent.z, k_sib);
    // without a child the record is dead (key 0) and its place is taken by the next one
    s.ent[f_cnt] = make_uint4(pack_lo(n, 0, d + 1, r_child),
                              (uint32_t)i_child | ((uint32_t)((d + 1) * k + r_child) << 15),
                              __float_as_uint(score), k_child);
#pragma unroll
    for (int q = 0; q < SLOTS; ++q) {
      fk[q] = (lane == wl && q == ws) ? k_sib : fk[q];
      fk[q] = (has_child && lane == cl && q == cs) ? k_child : fk[q];
    }
    if (LAZY) {  // fetch ahead the rows the two new records would open (unless they are open already)
      const int q_sib = d * k + r_sib, q_child = (d + 1) * k + r_child;
      if (has_sib && d < L && s.rowmap[q_sib] < 0) prefetch_row(s, src, q_sib, e_idx, k, L, lane);
      if (has_child && d + 1 < L && s.rowmap[q_child] < 0) prefetch_row(s, src, q_child, f_cnt, k, L, lane);
    }
    f_cnt += has_child ? 1 : 0;
    __syncwarp();
  }
  __syncwarp();
  return n_acc;
}

// ---------------------------------------------------------------------------- parallel expansion
// Exclusive prefix sum of one int per thread over the CTA (two barriers); `total` is the sum.
template <int T>
__device__ __forceinline__ int block_excl_scan(int v, Span<int> wsum, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += up;
  }
  if (lane == 31) wsum[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < T / 32; ++w) {
    const int x = wsum[w];
    base += w < warp ? x : 0;
    tot += x;
  }
  __syncthreads();
  total = tot;
  return base + inc - v;
}

// Is enumerated node a before node b in the total order, given equal scores and equal depths?  Token ascending,
// then the rank paths in lexicographic order (the candidates of a position are distinct tokens, so equal tokens
// mean equal last ranks and the paths differ higher up).
__device__ __forceinline__ bool tie_before(const TreeSmem& s, int a, int b, int k) {
  const int d = s.x_depth[a];
  const int ta = s.tok[(d - 1) * k + s.x_rank[a]], tb = s.tok[(d - 1) * k + s.x_rank[b]];
  if (ta != tb) return ta < tb;
  int ra = 0, rb = 0;
  while (a != b) {
    ra = s.x_rank[a]; rb = s.x_rank[b];
    a = s.x_parent[a]; b = s.x_parent[b];
  }
  return ra < rb;
}

// Algorithm 1 without a chain of N - 1 dependent pops: threshold rounds by one warp, then the final choice by
// the whole CTA.
//
// Scores never increase from a node to its children or to its later siblings (rows are sorted), so for any
// threshold the nodes that reach it form a set closed under "parent" and "earlier sibling" that can be
// enumerated in parallel: every enumerated node (one per lane) counts how many of its next children reach the
// threshold and appends them; the appended nodes do the same, wave after wave.  A round picks its threshold
// among the ordering keys of the nodes' best not-yet-enumerated children -- roughly the m-th best, with m the
// budget still open but at most half of those children (their keys are spread widely; the worst would pull in
// far more than the budget has room for) -- so a round adds at least one node and usually about doubles the
// set.  The threshold only steers how fast the set grows; the result does not depend on it: once at least
// `budget` nodes are enumerated (or nothing is left), every node outside the set scores below every node
// inside, the nodes of all rounds but the last beat those of the last, and the best of the last round under the
// total order fill the remaining places (eq. 12).
// Finite width (eq. 11): F_d = Top_W(E_d) holds the W best children of F_{d-1}, and nodes of earlier rounds beat
// those of later rounds, so a round sweeps the depths in order and, where a depth would exceed W, keeps only
// the best of its new candidates and closes the depth; the set is then F restricted to the threshold.
//
// expand_rounds_warp returns the number of enumerated nodes (root included; x_* arrays) and in `n_sure` how
// many of them precede the last round, or -1 if the set outgrew its capacity even for the smallest step
// (masses of exactly tied scores): the caller then falls back to the sequential search.
__device__ __forceinline__ int expand_rounds_warp(TreeSmem& s, int L, int k, int budget, int W, float zeta, int lane, int& n_sure) {
  const bool capped = W > 0 && W < budget;
  const int cap = s.xcap;
  if (lane == 0) {
    s.x_parent[0] = -1; s.x_depth[0] = 0; s.x_rank[0] = 0; s.x_next[0] = 0; s.x_score[0] = 0.f;
  }
  __syncwarp();
  int n = 1, shrink = 0;
  n_sure = 1;
  // every round that is not taken back adds a node, and a round is taken back at most a few times
  for (int guard = 0; budget - (n - 1) > 0; ++guard) {
    if (guard > 16 * (budget + 16)) return -1;
    const int remaining = budget - (n - 1);
    // ---- ordering key of every node's best child not yet enumerated (0 = none)
    int live = 0;
    uint32_t kmax = 0u;
    for (int i = lane; i < n; i += 32) {
      const int d = s.x_depth[i], j = s.x_next[i];
      uint32_t key = 0u;
      if (d < L && j < k && (!capped || s.depth_cnt[d + 1] < W)) {
        key = f2key(s.x_score[i] + s.t[(d * k + (int)s.x_rank[i]) * k + j] + zeta);
        key = key == 0u ? 1u : key;
      }
      s.x_key[i] = key;
      s.x_bak[i] = (unsigned char)j;
      live += key != 0u;
      kmax = key > kmax ? key : kmax;
    }
    live = __reduce_add_sync(FULL, live);
    kmax = __reduce_max_sync(FULL, kmax);
    if (live == 0) break;
    if (capped) for (int i = lane; i < L + 2; i += 32) s.depth_off[i] = s.depth_cnt[i];  // backup for a retry
    __syncwarp();
    // ---- threshold: the m-th best key, exactly while the set has at most 32 nodes, from 32 evenly spaced
    // nodes beyond that
    const int half = (live + 1) >> 1;
    int m = (remaining < half ? remaining : half) >> (2 * shrink);
    m = m < 1 ? 1 : m;
    uint32_t tau;
    {
      const int idx = n <= 32 ? lane : (lane * n) >> 5;
      const uint32_t mine = idx < n ? s.x_key[idx] : 0u;
      const int ls = __popc(__ballot_sync(FULL, mine != 0u));
      int r = 0;
#pragma unroll 8
      for (int j = 0; j < 32; ++j) {
        const uint32_t kj = __shfl_sync(FULL, mine, j);
        r += (kj > mine) || (kj == mine && j < lane);
      }
      int want = ls > 0 ? (m * ls + live - 1) / live - 1 : 0;
      want = want < 0 ? 0 : (want > ls - 1 ? ls - 1 : want);
      const unsigned holder = __ballot_sync(FULL, mine != 0u && r == want);
      tau = holder ? __shfl_sync(FULL, mine, __ffs(holder) - 1) : kmax;
    }
    const int n_before = n;
    bool overflow = false;
    // The qualifying children of node i, then those of the first child appended, and so on down: a chain of
    // best children costs one wave instead of one per level (the other new children wait for the next wave).
    // With `one` only node i's own children are taken (the depth sweep needs one depth at a time).
    auto chain = [&](int i, int at, bool write, bool one) {
      int d = s.x_depth[i], r = s.x_rank[i], j0 = s.x_next[i], par = i, total = 0;
      float sc = s.x_score[i];
      while (d < L) {
        const int base = (d * k + r) * k;
        int c = 0;
        while (j0 + c < k && f2key(sc + s.t[base + j0 + c] + zeta) >= tau) ++c;
        if (c == 0) break;
        if (write) {
          for (int q = 0; q < c; ++q) {
            const int idx = at + q;
            s.x_parent[idx] = (short)par; s.x_depth[idx] = (unsigned char)(d + 1);
            s.x_rank[idx] = s.ord[base + j0 + q]; s.x_score[idx] = sc + s.t[base + j0 + q] + zeta;
            s.x_next[idx] = 0;
          }
          s.x_next[par] = (unsigned char)(j0 + c);
        }
        total += c;
        if (one) break;
        sc = sc + s.t[base + j0] + zeta; r = s.ord[base + j0];
        par = at; at += c; d += 1; j0 = 0;
      }
      return total;
    };
    // one batch of 32 nodes: lane `mine` appends; returns false on overflow
    auto batch = [&](int i, bool mine, bool one) {
      const int c = mine ? chain(i, 0, false, one) : 0;
      int inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += up;
      }
      const int total = __shfl_sync(FULL, inc, 31);
      if (n + total > cap) return false;
      if (c) chain(i, n + inc - c, true, one);
      n += total;
      return true;
    };
    if (!capped) {
      int lo = 0, hi = n;
      bool first = true;
      while (true) {
        const int n_wave = n;
        for (int i0 = lo; i0 < hi && !overflow; i0 += 32) {
          const int i = i0 + lane;
          const bool mine = i < hi && (!first || (s.x_key[i] != 0u && s.x_key[i] >= tau));
          if (!__any_sync(FULL, mine)) continue;
          overflow = !batch(i, mine, false);
        }
        __syncwarp();  // the appended nodes are visible to every lane
        if (overflow || n == n_wave) break;
        lo = n_wave; hi = n; first = false;
      }
    } else {
      for (int d = 1; d <= L && !overflow; ++d) {
        const int room = W - s.depth_cnt[d];
        const int n_d = n;  // nodes [0, n_d) are the possible parents; candidates go to [n_d, ...)
        if (room <= 0) continue;
        for (int i0 = 0; i0 < n_d && !overflow; i0 += 32) {
          const int i = i0 + lane;
          const bool mine = i < n_d && (int)s.x_depth[i] == d - 1;
          if (!__any_sync(FULL, mine)) continue;
          overflow = !batch(i, mine, true);
        }
        __syncwarp();
        if (overflow) break;
        const int total_d = n - n_d;
        if (total_d > room) {
          // rank the candidates of this depth among themselves (score desc, token asc, rank path asc)
          for (int c = n_d + lane; c < n; c += 32) {
            const uint32_t kc = f2key(s.x_score[c]);
            int r = 0;
            for (int j = n_d; j < n; ++j) {
              const uint32_t kj = f2key(s.x_score[j]);
              r += (kj > kc) || (kj == kc && j != c && tie_before(s, j, c, k));
            }
            s.x_aux[c] = (short)(r < room ? 1 : 0);
          }
          __syncwarp();
          // stable compaction of the kept candidates to [n_d, n_d + room): destinations never pass sources
          int moved = 0;
          for (int c0 = n_d; c0 < n; c0 += 32) {
            const int c = c0 + lane;
            const int keep = c < n ? (int)s.x_aux[c] : 0;
            short cp = 0; unsigned char cr = 0; float cs = 0.f;
            if (keep) { cp = s.x_parent[c]; cr = s.x_rank[c]; cs = s.x_score[c]; }
            const unsigned kept = __ballot_sync(FULL, keep);
            __syncwarp();
            if (keep) {
              const int dst = n_d + moved + __popc(kept & ((1u << lane) - 1));
              s.x_parent[dst] = cp; s.x_rank[dst] = cr; s.x_score[dst] = cs;
              s.x_depth[dst] = (unsigned char)d; s.x_next[dst] = 0;
            }
            moved += __popc(kept);
            __syncwarp();
          }
          n = n_d + room;
          if (lane == 0) s.depth_cnt[d] = W;
        } else if (lane == 0) {
          s.depth_cnt[d] += total_d;
        }
        __syncwarp();
      }
    }
    if (overflow) {
      if (m == 1) return -1;
      for (int i = lane; i < n_before; i += 32) s.x_next[i] = s.x_bak[i];
      if (capped) for (int i = lane; i < L + 2; i += 32) s.depth_cnt[i] = s.depth_off[i];
      n = n_before;
      ++shrink;
      __syncwarp();
      continue;
    }
    shrink = 0;
    n_sure = n_before;
  }
  return n;
}

// The same rounds by EX_T threads (four warps; the others wait at the CTA barrier behind the call), for an
// unbounded width: no depth needs closing, so nodes may be appended in any order -- one thread per node, places in
// the node arrays reserved with a shared counter, two barriers per wave.  The order of the nodes in the arrays
// then varies from run to run; the result does not (the final choice and the slot layout depend on scores,
// depths and rank paths only).
// Threshold of a round: the rank rule of expand_rounds_warp on 32 evenly spaced nodes, lowered further, from the
// third round on, to where the count of enumerated nodes -- which grows roughly geometrically as the threshold
// falls -- is expected to pass the budget (a secant step on log(count) over the last two thresholds).  A round
// that outgrows the node arrays is taken back and repeated with a smaller step.
// scalars[1] = node count, scalars[2] = threshold key, scalars[3] = flags (1: nothing left, 2: out of room,
// 4: smallest step).
constexpr int EX_T = 128;
constexpr float kFirstShare = 1.5f;  // first threshold of the rounds: path probability kFirstShare / budget
__device__ __forceinline__ void ex_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(EX_T) : "memory"); }

__device__ __forceinline__ void prepare_rows(TreeSmem& s, int k, int row0, int nrows, int tid, int nthreads);
__device__ __forceinline__ int expand_rounds_cta(TreeSmem& s, int L, int k, int budget, float zeta, int& n_sure,
                                                 int& d_ready) {
  const int tid = threadIdx.x, lane = tid & 31;
  const int cap = s.xcap;
  if (tid == 0) {
    s.x_parent[0] = -1; s.x_depth[0] = 0; s.x_rank[0] = 0; s.x_next[0] = 0; s.x_score[0] = 0.f;
    s.scalars[1] = 1;
    s.scalars[3] = 0;
  }
  ex_barrier();
  int n = 1, shrink = 0;
  n_sure = 1;
  // ordering key of node i's best child not yet enumerated, 0 = none
  auto open_key = [&](int i) -> uint32_t {
    const int d = s.x_depth[i], j = s.x_next[i];
    if (d >= L || j >= k) return 0u;
    const uint32_t key = f2key(s.x_score[i] + s.t[(d * k + (int)s.x_rank[i]) * k + j] + zeta);
    return key == 0u ? 1u : key;
  };
  float t_prev = 0.f, t_prev2 = 0.f;  // thresholds of the last two rounds that stood (warp 0 only)
  int n_prev = 0, n_prev2 = 0;        // ... and the node counts they led to
  for (int guard = 0; budget - (n - 1) > 0; ++guard) {
    if (guard > 16 * (budget + 16)) return -1;
    const int remaining = budget - (n - 1);
    uint32_t tau = 0u;
    bool smallest_step = false;
    if (guard == 0) {
      // First round (only the root is there): the successor scores of a row are normalised (eq. 9), so a node's
      // score is the logarithm of a path probability (plus depth * zeta <= 0) and at most 1 / theta nodes of a depth
      // reach ln theta: start at theta = kFirstShare / budget instead of at the best child of the root.  Every
      // thread computes it; no barrier.
      const uint32_t kbest = open_key(0);
      if (kbest == 0u) break;
      uint32_t k1 = f2key(-__logf((float)budget * (1.0f / kFirstShare)));
      k1 = k1 == 0u ? 1u : k1;
      tau = k1 < kbest ? k1 : kbest;  // a round must add at least the best open child
    } else {
      if (tid < 32) {
        const int idx = n <= 32 ? lane : (lane * n) >> 5;
        const uint32_t mine = idx < n ? open_key(idx) : 0u;
        int ls = __popc(__ballot_sync(FULL, mine != 0u));
        uint32_t kmax = __reduce_max_sync(FULL, mine);
        int live = n <= 32 ? ls : (ls * n + 31) >> 5;  // beyond 32 nodes an estimate is all the rule needs
        if (ls == 0 && n > 32) {                       // none in the sample: look at every node
          int cnt = 0;
          for (int i = lane; i < n; i += 32) {
            const uint32_t key = open_key(i);
            cnt += key != 0u;
            kmax = key > kmax ? key : kmax;
          }
          live = __reduce_add_sync(FULL, cnt);
          kmax = __reduce_max_sync(FULL, kmax);
        }
        const int half = (live + 1) >> 1;
        int m = (remaining < half ? remaining : half) >> (2 * shrink);
        m = m < 1 ? 1 : m;
        int r = 0;
  #pragma unroll 8
        for (int j = 0; j < 32; ++j) {
          const uint32_t kj = __shfl_sync(FULL, mine, j);
          r += (kj > mine) || (kj == mine && j < lane);
        }
        int want = ls > 0 ? (m * ls + live - 1) / (live > 0 ? live : 1) - 1 : 0;
        want = want < 0 ? 0 : (want > ls - 1 ? ls - 1 : want);
        const unsigned holder = __ballot_sync(FULL, mine != 0u && r == want);
        tau = holder ? __shfl_sync(FULL, mine, __ffs(holder) - 1) : kmax;
        if (shrink == 0 && n_prev2 >= 8 && n_prev > n_prev2 && t_prev < t_prev2) {
          // secant step, never below the key that the rank rule gives for the whole open budget
          int mf = remaining < live ? remaining : live;
          int wf = ls > 0 ? (mf * ls + live - 1) / (live > 0 ? live : 1) - 1 : 0;
          wf = wf < 0 ? 0 : (wf > ls - 1 ? ls - 1 : wf);
          const unsigned hf = __ballot_sync(FULL, mine != 0u && r == wf);
          const uint32_t tau_full = hf ? __shfl_sync(FULL, mine, __ffs(hf) - 1) : tau;
          const float ln1 = __logf((float)n_prev2), ln2 = __logf((float)n_prev);
          const float slope = (ln2 - ln1) / (t_prev2 - t_prev);
          const float ts = t_prev - (__logf((float)(budget + 1)) - ln2) / slope;
          if (ts == ts && ts < 0.f) {
            uint32_t ks = f2key(ts);
            ks = ks == 0u ? 1u : ks;
            ks = ks < tau_full ? tau_full : ks;
            tau = ks < tau ? ks : tau;
          }
        }
        if (tau > kmax) tau = kmax;  // a round must add at least the best open child
        if (lane == 0) {
          s.scalars[2] = (int)tau;
          s.scalars[3] = (live == 0 || kmax == 0u ? 1 : 0) | (m == 1 && shrink > 0 ? 4 : 0);
        }
      }
      ex_barrier();
      if (s.scalars[3] & 1) break;
      smallest_step = (s.scalars[3] & 4) != 0;
      tau = (uint32_t)s.scalars[2];
    }
    const int n_before = n;
    // The children of node i that reach the threshold (a row is sorted: they are the next ones in it); they
    // reserve their places with the shared counter and are visited themselves in the next wave.  (Walking on down
    // the first child in the same wave was measured: the long serial chains cost more than the waves they save
    // once a round adds dozens of nodes.)
    auto chain = [&](int i) {
      const int d = s.x_depth[i];
      if (d >= L) return;
      const int j0 = s.x_next[i], base = (d * k + (int)s.x_rank[i]) * k;
      const float sc = s.x_score[i];
      int c = 0;
      while (j0 + c < k && f2key(sc + s.t[base + j0 + c] + zeta) >= tau) ++c;
      if (c == 0) return;
      const int at = atomicAdd(&s.scalars[1], c);
      if (at + c > cap) { atomicOr(&s.scalars[3], 2); return; }
      for (int q = 0; q < c; ++q) {
        const int idx = at + q;
        s.x_parent[idx] = (short)i; s.x_depth[idx] = (unsigned char)(d + 1);
        s.x_rank[idx] = s.ord[base + j0 + q]; s.x_score[idx] = sc + s.t[base + j0 + q] + zeta;
        s.x_next[idx] = 0;
      }
      s.x_next[i] = (unsigned char)(j0 + c);
      // the children just appended open rows that are not prepared yet
      if (d + 1 >= d_ready && d_ready < L) atomicOr(&s.scalars[3], 8);
    };
    int lo = 0, hi = n;
    bool first = true, overflow = false;
    while (true) {
      for (int i = lo + tid; i < hi; i += EX_T) {
        if (first) s.x_bak[i] = s.x_next[i];  // for taking the round back
        chain(i);
      }
      ex_barrier();  // the appended nodes and the counter are final for this wave
      const int n_now = s.scalars[1];
      overflow = (s.scalars[3] & 2) != 0;
      const bool deeper = (s.scalars[3] & 8) != 0;
      ex_barrier();  // ... and every thread has read them before the next wave moves them on
      if (deeper && d_ready < L) {  // a node beyond the prepared positions: prepare the rest of the table now
        prepare_rows(s, k, 1 + (d_ready - 1) * k, 1 + (L - 1) * k, tid, EX_T);
        d_ready = L;
        ex_barrier();
      }
      if (overflow || n_now == hi) { n = n_now; break; }
      lo = hi; hi = n_now; first = false;
      n = n_now;
    }
    if (overflow) {
      if (smallest_step) return -1;
      for (int i = tid; i < n_before; i += EX_T) s.x_next[i] = s.x_bak[i];
      if (tid == 0) { s.scalars[1] = n_before; s.scalars[3] = 0; }
      n = n_before;
      ++shrink;
      ex_barrier();
      continue;
    }
    shrink = 0;
    n_sure = n_before;
    t_prev2 = t_prev; n_prev2 = n_prev;
    t_prev = key2f(tau); n_prev = n;
  }
  return n;
}

// The `budget` best of the enumerated nodes under the total order, compacted into nd_*; every thread of the
// CTA calls it.  Nodes [1, n_sure) come from earlier rounds than [n_sure, n) and beat them all, so only the
// nodes of the last round compete, for the places the earlier ones leave open.  Returns the number selected.
template <int T>
__device__ __forceinline__ int select_enumerated(TreeSmem& s, int n, int n_sure, int budget, int k) {
  const int tid = threadIdx.x;
  const bool all = n - 1 <= budget;
  const int places = budget - (n_sure - 1);
  if (!all) {  // ordering keys of the competitors: (score, depth ascending)
    for (int i = n_sure + tid; i < n; i += T)
      s.x_key64[i] = ((uint64_t)f2key(s.x_score[i]) << 32) | (uint32_t)(255 - (int)s.x_depth[i]);
  }
  __syncthreads();
  int n_sel = 0;
  for (int i0 = 1; i0 < n; i0 += T) {
    const int i = i0 + tid;
    int sel = 0;
    if (i < n) {
      sel = 1;
      if (!all && i >= n_sure) {
        const uint64_t ki = s.x_key64[i];
        int r = 0, eq = 0;
#pragma unroll 4
        for (int j = n_sure; j < n; ++j) {
          const uint64_t kj = s.x_key64[j];
          r += kj > ki;
          eq += kj == ki;
        }
        if (eq > 1 && r < places)  // exactly tied scores at one depth (rare): token, then rank path decide
          for (int j = n_sure; j < n; ++j) r += s.x_key64[j] == ki && j != i && tie_before(s, j, i, k);
        sel = r < places;
      }
    }
    int total;
    const int off = block_excl_scan<T>(sel, s.x_wsum, total);
    if (i < n) s.x_aux[i] = (short)(sel ? n_sel + off : -1);
    n_sel += total;
  }
  __syncthreads();
  for (int i = 1 + tid; i < n; i += T) {
    const int at = s.x_aux[i];
    if (at < 0) continue;
    const int p = s.x_parent[i];
    s.nd_parent[at] = (short)(p == 0 ? -1 : s.x_aux[p]);
    s.nd_depth[at] = s.x_depth[i];
    s.nd_rank[at] = s.x_rank[i];
    s.nd_score[at] = s.x_score[i];
  }
  __syncthreads();
  return n_sel;
}

// Eq. 11 as it stands, for the case the other forms serve badly: the pair table does not fit in shared memory
// (k = 64) and the width is small (W <= 16).  Depth by depth: one warp per node of F_{d-1} fetches the raw selector
// scores of the node's row from global memory, applies eq. 5 and eq. 9 with the row in registers (two successors
// per lane) and extracts the row's min(W, k) best children under (score desc, token asc) -- no other child of
// that node can be among the W best of the depth; then all threads rank the at most W * W candidates of the depth
// under the total order, and the W best become F_d.  The node arrays end up holding S = F_1 u ... u F_L (root at
// 0); the caller picks the budget's best of them (eq. 12).  Two CTA barriers per depth, and the only dependent
// global access per depth is one 4 k-byte row per node, so the chain is L short steps instead of N - 1 pops that
// each prepare a row.  Every thread of the CTA calls this; returns the number of enumerated nodes, root included.
__device__ __forceinline__ int expand_depthwise(TreeSmem& s, const RowSource& src, int L, int k, int W, float zeta) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int NW = G2_T / 32;
  const int m = W < k ? W : k;      // children a node can contribute to its depth
  const int cbase = 1 + W * L;      // candidates of the current depth live behind the nodes
  if (tid == 0) { s.x_parent[0] = -1; s.x_depth[0] = 0; s.x_rank[0] = 0; s.x_score[0] = 0.f; }
  __syncthreads();
  int lo = 0, hi = 1;               // F_{d-1} = nodes [lo, hi)
  for (int d = 1; d <= L; ++d) {
    const int np = hi - lo, i = d - 1;  // i: position of the children
    const float al = s.al[i], la = s.la[i];
    for (int p = warp; p < np; p += NW) {
      const int node = lo + p, ra = d == 1 ? 0 : (int)s.x_rank[node];
      const float sc = s.x_score[node];
      const float* row = i == 0 ? src.anchor_bigram : src.bigram + ((size_t)(i - 1) * k + ra) * k;
      float v[2];
      uint32_t ntok[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int rb = lane + 32 * h;
        v[h] = -INFINITY;
        ntok[h] = 0u;
        if (rb < k) {
          v[h] = fmaf(al, s.lp[i * k + rb], la * (row ? __ldg(row + rb) : 0.f));
          ntok[h] = ~(uint32_t)s.tok[i * k + rb];
        }
      }
      float mx = fmaxf(v[0], v[1]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
      float sum = (lane < k ? expf(v[0] - mx) : 0.f) + (lane + 32 < k ? expf(v[1] - mx) : 0.f);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
      const float lse = mx + logf(sum);
      // the children's scores, ranked within the row; those with fewer than m in front become candidates of the
      // depth at the place of that rank
#pragma unroll
      for (int h = 0; h < 2; ++h) v[h] = sc + (v[h] - lse) + zeta;
      unsigned long long k64[2];
      int r0, r1;
      rank_row_warp(s, v, ntok, k, lane, k64, r0, r1);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int rb = lane + 32 * h, r = h == 0 ? r0 : r1;
        if (rb < k && r < m) {
          const int c = cbase + p * m + r;
          s.x_parent[c] = (short)node;
          s.x_rank[c] = (unsigned char)rb;
          s.x_score[c] = v[h];
          s.x_key64[c] = k64[h];
          s.dw_ckey[p * m + r] = (uint32_t)(k64[h] >> 32);
          if (d < L && src.bigram) {  // the row this child would open at the next depth: start fetching it now, the
            const float* nxt = src.bigram + ((size_t)(d - 1) * k + rb) * k;  // ranking below covers the latency
            asm volatile("prefetch.global.L1 [%0];" ::"l"(nxt));
            if (k > 32) asm volatile("prefetch.global.L1 [%0];" ::"l"(nxt + 32));
          }
        }
      }
      __syncwarp();
    }
    __syncthreads();
    // the W best of the depth's candidates under (score desc, token asc, rank path asc): `sp` threads share the
    // count of one candidate; the loop is branch-free, exact ties (rare) are settled behind it
    const int nc = np * m;
    int sp = 1;
    while (sp < 8 && sp * 2 * nc <= G2_T) sp <<= 1;
    const int cand = tid / sp, q = tid & (sp - 1);
    int r = 0, same = 0;
    unsigned long long kc = 0ull;
    if (cand < nc) {
      kc = s.x_key64[cbase + cand];
      const uint32_t sc32 = (uint32_t)(kc >> 32);  // the loop compares score keys only, four per load
      const uint4* ck = reinterpret_cast<const uint4*>(s.dw_ckey.ptr(0, (nc + 3) & ~3));
      const int n4 = nc >> 2;
      int c0 = 0, c1 = 0, c2 = 0, c3 = 0, e0 = 0, e1 = 0, e2 = 0, e3 = 0;  // independent counters (see rank_row_warp)
#pragma unroll 4
      for (int j = q; j < n4; j += sp) {
        const uint4 w = ck[j];
        c0 += w.x > sc32; c1 += w.y > sc32; c2 += w.z > sc32; c3 += w.w > sc32;
        e0 += w.x == sc32; e1 += w.y == sc32; e2 += w.z == sc32; e3 += w.w == sc32;
      }
      r = (c0 + c1) + (c2 + c3);
      same = (e0 + e1) + (e2 + e3);
      if (q == 0)
        for (int j = n4 * 4; j < nc; ++j) {  // the last one to three
          const uint32_t kj = s.dw_ckey[j];
          r += kj > sc32;
          same += kj == sc32;
        }
    }
    for (int o = sp >> 1; o > 0; o >>= 1) {
      r += __shfl_xor_sync(FULL, r, o);
      same += __shfl_xor_sync(FULL, same, o);
    }
    if (cand < nc && q == 0) {
      if (same > 1) {  // equal scores (rare): the token decides, then the parents' rank paths
        for (int j = 0; j < nc; ++j) {
          const unsigned long long kj = s.x_key64[cbase + j];
          if (j == cand || (uint32_t)(kj >> 32) != (uint32_t)(kc >> 32)) continue;
          if (kj != kc) { r += kj > kc; continue; }
          int a = s.x_parent[cbase + j], bnode = s.x_parent[cbase + cand], ra2 = 0, rb2 = 0;
          while (a != bnode) {
            ra2 = s.x_rank[a]; rb2 = s.x_rank[bnode];
            a = s.x_parent[a]; bnode = s.x_parent[bnode];
          }
          r += ra2 < rb2;
        }
      }
      if (r < W) {
        const int at = hi + r, rk = s.x_rank[cbase + cand];
        s.x_parent[at] = s.x_parent[cbase + cand];
        s.x_depth[at] = (unsigned char)d;
        s.x_rank[at] = (unsigned char)rk;
        s.x_score[at] = s.x_score[cbase + cand];
      }
    }
    __syncthreads();
    lo = hi;
    hi += nc < W ? nc : W;
  }
  return hi;
}

// eq. 5 and eq. 9, then the sort by (t desc, token asc), one THREAD per (position, predecessor) row, for k <= KP
// <= 4: the row lives in registers, nothing is exchanged between lanes and the k^2 comparisons are independent
// of one another.  Element e of the row is visited in an order that starts at tid % k, so that the lanes of a
// warp spread over the shared-memory banks.  In place: a thread reads its whole row before it rewrites it.
template <int KP>
__device__ __forceinline__ void prepare_rows_by_thread(TreeSmem& s, int k, int row0, int nrows, int tid, int nthreads) {
  const int start = tid % k;
  for (int r = row0 + tid; r < nrows; r += nthreads) {
    const int i = r == 0 ? 0 : 1 + (r - 1) / k;
    const int ra = r == 0 ? 0 : (r - 1) % k;
    const int at = (i * k + ra) * k;
    const float al = s.al[i];
    float v[KP];
    int tk[KP];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < KP; ++j) {
      int e = start + j;
      e = e >= k ? e - k : e;
      v[j] = -INFINITY;
      tk[j] = 0;
      if (j < k) {
        v[j] = fmaf(al, s.lp[i * k + e], s.t[at + e]);
        tk[j] = s.tok[i * k + e];
        mx = fmaxf(mx, v[j]);
      }
    }
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < KP; ++j) sum += j < k ? expf(v[j] - mx) : 0.f;
    const float lse = mx + logf(sum);
    unsigned long long key[KP];  // (value desc, token asc) as one descending key
#pragma unroll
    for (int j = 0; j < KP; ++j) {
      v[j] -= lse;
      key[j] = ((unsigned long long)f2key(v[j]) << 32) | (uint32_t)(~(uint32_t)tk[j]);
    }
#pragma unroll
    for (int a = 0; a < KP; ++a) {
      if (a >= k) break;
      int rank = 0;
#pragma unroll
      for (int c = 0; c < KP; ++c)
        if (c < k) rank += (key[c] > key[a]) || (key[c] == key[a] && c < a);  // equal keys: a permutation all the same
      int e = start + a;
      e = e >= k ? e - k : e;
      s.t[at + rank] = v[a];
      s.ord[at + rank] = (unsigned char)e;
    }
  }
}

// The same for 8 <= KP <= 16 (KP a power of two, k <= KP): KP lanes per row, 32 / KP rows per warp at a time, one entry
// per lane.  The log-sum-exp is a butterfly inside the lane group; the ranks come from counting the group's 32-bit
// value keys out of the warp's scratch (KP / 4 vector loads per lane), with the same collision check and 64-bit
// recount for equal values as rank_row_warp.  A thread that holds a whole row of 16 in registers spends a thousand
// dependent instructions on it while most of the CTA's issue slots stay empty; here a row costs a few dozen.
template <int KP>
__device__ __forceinline__ void prepare_rows_by_group(TreeSmem& s, int k, int row0, int nrows, int tid, int nthreads) {
  constexpr int RPW = 32 / KP;
  const int lane = tid & 31, warp = tid >> 5, g = lane / KP, e = lane % KP;
  unsigned long long* scratch64 = s.dw_row.ptr((long long)warp * 32, 32);
  uint32_t* key32 = reinterpret_cast<uint32_t*>(scratch64);  // [32] value keys (0 = none), then [32] marks
  for (int rbase = row0 + warp * RPW; rbase < nrows; rbase += (nthreads / 32) * RPW) {
    const int r = rbase + g;
    const bool on = r < nrows && e < k;
    const int i = r == 0 ? 0 : 1 + (r - 1) / k;
    const int ra = r == 0 ? 0 : (r - 1) % k;
    const int at = (i * k + ra) * k;
    float v = -INFINITY;
    uint32_t ntok = 0u;
    if (on) {
      v = fmaf(s.al[i], s.lp[i * k + e], s.t[at + e]);
      ntok = ~(uint32_t)s.tok[i * k + e];
    }
    float mx = v;
#pragma unroll
    for (int o = KP / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
    float sum = on ? expf(v - mx) : 0.f;
#pragma unroll
    for (int o = KP / 2; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
    v -= mx + logf(sum);
    uint32_t kv = f2key(v);
    kv = kv == 0u ? 1u : kv;
    key32[lane] = on ? kv : 0u;
    __syncwarp();
    const uint4* grp = reinterpret_cast<const uint4*>(key32 + g * KP);
    int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
#pragma unroll
    for (int j = 0; j < KP / 4; ++j) {
      const uint4 q = grp[j];
      c0 += q.x > kv; c1 += q.y > kv; c2 += q.z > kv; c3 += q.w > kv;
    }
    int rank = (c0 + c1) + (c2 + c3);
    if (on) key32[32 + g * KP + rank] = (uint32_t)e;
    __syncwarp();
    const bool clash = on && key32[32 + g * KP + rank] != (uint32_t)e;
    if (__any_sync(FULL, clash)) {  // equal values in a row: rank again on (value key, ~token)
      __syncwarp();
      const unsigned long long k64 = ((unsigned long long)kv << 32) | ntok;
      scratch64[lane] = on ? k64 : 0ull;
      __syncwarp();
      rank = 0;
      for (int j = 0; j < k; ++j) rank += scratch64[g * KP + j] > k64;
    }
    __syncwarp();  // every lane has read its raw entry and the scratch: both may be rewritten
    if (on) {
      s.t[at + rank] = v;
      s.ord[at + rank] = (unsigned char)e;
    }
  }
}

// Rows [row0, nrows) of a table of k <= 16 successors per row, by the first `nthreads` threads of the CTA (a
// multiple of 32; all of them call).
__device__ __forceinline__ void prepare_rows(TreeSmem& s, int k, int row0, int nrows, int tid, int nthreads) {
  if (k <= 1) prepare_rows_by_thread<1>(s, k, row0, nrows, tid, nthreads);
  else if (k <= 2) prepare_rows_by_thread<2>(s, k, row0, nrows, tid, nthreads);
  else if (k <= 4) prepare_rows_by_thread<4>(s, k, row0, nrows, tid, nthreads);
  else if (k <= 8) prepare_rows_by_group<8>(s, k, row0, nrows, tid, nthreads);
  else prepare_rows_by_group<16>(s, k, row0, nrows, tid, nthreads);
}
// With k <= 16 and unbounded width the rows of the first kEagerDepths positions are prepared up front and the
// rest only if the expansion appends a node that deep: a budget of a few hundred nodes rarely reaches beyond
// depth 12, while the positions go up to L = 32.
constexpr int kEagerDepths = 16;

// LAZY: the rows of the pair table are computed on demand (see TreeSmem).
template <bool LAZY>
__global__ void __launch_bounds__(G2_T, 1)
k_build_tree(const float* __restrict__ bigram, int L, int k, int N, int W, float zeta,
             const float* __restrict__ alpha, const float* __restrict__ lambda,
             const float* __restrict__ anchor_bigram, const int32_t* __restrict__ anchor_tokens,
             const int32_t* __restrict__ pos_offset, ubt_tree out, MergeParts parts, int V,
             int32_t* __restrict__ status, const __grid_constant__ TreeLayout lay) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TreeSmem s;
  tree_bind(&s, smem_raw, lay, L, k, N);
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const int kk2 = k * k, mw = (N + 31) / 32, budget = N - 1;
  const long long nB = gridDim.x;
  const Span<const float> g_lp(out.cand_logprob, nB * L * k, 201), g_big(bigram, nB * (L - 1) * kk2, 203);
  const Span<const int32_t> g_ids(out.cand_ids, nB * L * k, 202);
  const Span<int32_t> g_tok(out.token_ids, nB * N, 211), g_par(out.parents, nB * N, 212), g_dep(out.depths, nB * N, 213);
  const Span<int32_t> g_rk(out.cand_rank, nB * N, 214), g_pos(out.position_ids, nB * N, 215), g_nn(out.n_nodes, nB, 216);
  const Span<float> g_sc(out.scores, nB * N, 217);
  const Span<uint32_t> g_mask(out.mask, nB * N * mw, 218);
  // The next kernel in the stream may start right away.  When that is the V-wide pass of ubt_verify_tree it
  // reads target logits only and streams while this kernel (and the tail of the top-k kernel in front of it)
  // is still running; it waits for this grid before it exits, so stream order still holds for whatever follows.
  // The host side launches it that way only if nothing it writes touches a buffer of this draft call; any
  // other kernel is launched normally and starts after this grid has completed, whatever is signalled here.
  pdl_launch_dependents();
  // ---- the selector's scores, scaled by eq. 5's lambda, go to shared memory first.  They are an input of
  // the call, complete before the streaming kernel ahead of this one was launched, so they may be read
  // while that kernel is still running: their DRAM latency hides behind its tail.
  const int nrows = 1 + (L - 1) * k;
  constexpr bool lazy = LAZY;
  for (int i = tid; i < L; i += G2_T) {
    s.al[i] = alpha ? alpha[i] : 1.f;
    s.la[i] = lambda ? lambda[i] : 1.f;
  }
  if (tid == 0) s.scalars[4] = 0;
  if constexpr (lazy) {
    for (int i = tid; i < L * k + 1; i += G2_T) s.rowmap[i] = (short)-1;
  } else {
    const int n_big = (L - 1) * kk2;
    constexpr int U = 8;
    for (int i0 = 0; i0 < n_big; i0 += G2_T * U) {
      float d[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * G2_T + tid;
        d[u] = i < n_big ? g_big[(int64_t)b * n_big + i] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u * G2_T + tid;
        if (i < n_big) s.t[kk2 + i] = (lambda ? lambda[1 + i / kk2] : 1.f) * d[u];
      }
    }
    for (int i = tid; i < kk2; i += G2_T)  // position 0: only predecessor row 0 exists
      s.t[i] = (i < k && anchor_bigram) ? (lambda ? lambda[0] : 1.f) * anchor_bigram[(int64_t)b * k + i] : 0.f;
  }
  pdl_wait();  // the partials / candidates come from the kernel before this one

  // ---- step a1's last part when fused: merge the row partials of this sequence's L rows (one warp per row; the
  // candidates go to global memory and to the shared-memory staging at once); otherwise stage the candidates
  if (parts.part_ms != nullptr) {
    for (int i = tid >> 5; i < L; i += G2_T / 32) {
      const int bits = merge_row_warp(parts, nB * L, (int64_t)b * L + i, V, k, out.cand_ids, out.cand_logprob, lane,
                                      s.tok.ptr((long long)i * k, k), s.lp.ptr((long long)i * k, k));
      if (bits && lane == 0) atomicOr(&s.scalars[4], bits);
    }
  } else {
    for (int i = tid; i < L * k; i += G2_T) {
      const float lpv = g_lp[(int64_t)b * L * k + i];
      s.lp[i] = lpv;
      s.tok[i] = g_ids[(int64_t)b * L * k + i];
      if (!(lpv <= 0.f || lpv > 0.f) || lpv == INFINITY) atomicOr(&s.scalars[4], kStatusNonFinite);
    }
  }
  // positions whose rows are prepared before the expansion starts (all of them unless the threshold rounds run)
  const bool rounds_cta = !LAZY && !(W > 0 && W < budget);
  int d_ready = rounds_cta && k <= 16 && L > kEagerDepths ? kEagerDepths : L;
  if constexpr (lazy) {
    // rows are normalised and sorted by the expanding warp, one at a time, when the search first needs them
  } else if (k <= 16) {
    __syncthreads();  // s.lp, s.tok
    prepare_rows(s, k, 0, 1 + (d_ready - 1) * k, tid, G2_T);
  } else {
    // 16 < k <= 64: one warp per (position, predecessor) row, two entries per lane; eq. 5, eq. 9, ranks by counting
    __syncthreads();  // s.lp, s.tok
    for (int r = tid >> 5; r < nrows; r += G2_T / 32) {
      const int i = r == 0 ? 0 : 1 + (r - 1) / k;
      const int ra = r == 0 ? 0 : (r - 1) % k;
      const int at = (i * k + ra) * k;
      const float al = s.al[i];
      float v[2];
      uint32_t ntok[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int rb = lane + 32 * h;
        v[h] = -INFINITY;
        ntok[h] = 0u;
        if (rb < k) {
          v[h] = fmaf(al, s.lp[i * k + rb], s.t[at + rb]);
          ntok[h] = ~(uint32_t)s.tok[i * k + rb];
        }
      }
      float mx = fmaxf(v[0], v[1]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
      float sum = (lane < k ? expf(v[0] - mx) : 0.f) + (lane + 32 < k ? expf(v[1] - mx) : 0.f);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
      const float lse = mx + logf(sum);
      v[0] -= lse; v[1] -= lse;
      unsigned long long k64[2];
      int r0, r1;
      rank_row_warp(s, v, ntok, k, lane, k64, r0, r1);  // (every lane has read its raw entries: the row may be rewritten)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int rb = lane + 32 * h, rk = h == 0 ? r0 : r1;
        if (rb < k) {
          s.t[at + rk] = v[h];
          s.ord[at + rk] = (unsigned char)rb;
        }
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < L + 2; i += G2_T) s.depth_cnt[i] = 0;
  for (int i = tid; i < N * mw; i += G2_T) s.maskrow[i] = 0u;
  __syncthreads();
  // ---- expansion: by the whole CTA when the table is resident; the sequential best-first search by one warp
  // serves the lazy mode and the rare inputs the parallel form gives up on
  int bits = 1;
  while ((1 << bits) < k) ++bits;
  const bool use_pk = bits * L <= 128;
  bool sequential = LAZY;
  RowSource src;
  src.bigram = L > 1 ? bigram + (size_t)b * (L - 1) * kk2 : nullptr;
  src.anchor_bigram = anchor_bigram ? anchor_bigram + (size_t)b * k : nullptr;
  if constexpr (LAZY) {
    if (s.xcap > 0) {  // a small finite width: eq. 11 depth by depth, then eq. 12 on the union
      const int n = expand_depthwise(s, src, L, k, W, zeta);
      const int n_sel = select_enumerated<G2_T>(s, n, 1, budget, k);
      if (tid == 0) s.scalars[0] = n_sel;
      sequential = false;
    }
  }
  if constexpr (!LAZY) {
    int n;
    if (W > 0 && W < budget) {  // a finite width closes depths in order: one warp
      if (tid < 32) {
        int n_sure = 1;
        const int nn = expand_rounds_warp(s, L, k, budget, W, zeta, lane, n_sure);
        if (lane == 0) { s.scalars[1] = nn; s.scalars[2] = n_sure; }
      }
      __syncthreads();
      n = s.scalars[1];
    } else {
      if (tid < EX_T) {
        int n_sure = 1;
        const int nn = expand_rounds_cta(s, L, k, budget, zeta, n_sure, d_ready);
        if (tid == 0) { s.scalars[1] = nn; s.scalars[2] = n_sure; s.scalars[5] = d_ready; }
      }
      __syncthreads();
      n = s.scalars[1];
      d_ready = s.scalars[5];
    }
    if (n < 0) {
      if (d_ready < L) {  // the sequential search may open any row
        prepare_rows(s, k, 1 + (d_ready - 1) * k, 1 + (L - 1) * k, tid, G2_T);
        d_ready = L;
      }
      sequential = true;
      for (int i = tid; i < L + 2; i += G2_T) s.depth_cnt[i] = 0;
      __syncthreads();
    } else {
      const int n_sel = select_enumerated<G2_T>(s, n, s.scalars[2], budget, k);
      if (tid == 0) s.scalars[0] = n_sel;
    }
  }
  if (sequential && tid < 32) {
    int n;
    if (N <= 64) n = expand_tree<2, LAZY>(s, src, L, k, budget, W, zeta, lane);
    else if (N <= 128) n = expand_tree<4, LAZY>(s, src, L, k, budget, W, zeta, lane);
    else n = expand_tree<8, LAZY>(s, src, L, k, budget, W, zeta, lane);
    if (lane == 0) s.scalars[0] = n;
  }
  __syncthreads();
  // ---- canonical slots: root 0, then depth by depth ordered by (parent slot, rank)
  const int n_acc = s.scalars[0];
  for (int i = tid; i < L + 2; i += G2_T) { s.depth_cnt[i] = 0; s.x_fill[i] = 0; }
  __syncthreads();
  if (tid < n_acc) {
    atomicAdd(&s.depth_cnt[s.nd_depth[tid]], 1);
    if (use_pk) {  // rank path packed big-endian: walk up to the root
      unsigned long long hi = 0ull, lo = 0ull;
      for (int a = tid; a >= 0; a = s.nd_parent[a]) {
        const int sh = 128 - bits * (int)s.nd_depth[a];
        const unsigned long long r = s.nd_rank[a];
        if (sh >= 64) {
          hi |= r << (sh - 64);
        } else {
          lo |= r << sh;
          if (sh + bits > 64) hi |= r >> (64 - sh);  // the field straddles the two words
        }
      }
      s.nd_pk[2 * tid] = hi; s.nd_pk[2 * tid + 1] = lo;
    }
  }
  __syncthreads();
  if (tid == 0) {
    int off = 1;
    for (int d = 1; d <= L; ++d) { s.depth_off[d] = off; off += s.depth_cnt[d]; }
  }
  __syncthreads();
  if (use_pk) {
    // inside a depth, (parent slot, rank) order is the lexicographic order of the rank paths.  The nodes are first
    // grouped by depth (kk = node indices, depth by depth), so that a node is compared with its own depth only;
    // the count for one node is shared by `sp` neighbouring lanes
    if (tid < n_acc) {
      const int d = s.nd_depth[tid];
      s.kk[s.depth_off[d] - 1 + atomicAdd(&s.x_fill[d], 1)] = tid;
    }
    __syncthreads();
    int sp = 1;
    while (sp < 32 && sp * 2 * n_acc <= 2 * G2_T && sp * 2 * n_acc > 0) sp <<= 1;
    if (sp * n_acc > G2_T) sp >>= 1;
    const int node = tid / sp, q = tid & (sp - 1);
    const bool mine = node < n_acc;
    const int d = mine ? s.nd_depth[node] : 0;
    const unsigned long long hi = mine ? s.nd_pk[2 * node] : 0ull, lo = mine ? s.nd_pk[2 * node + 1] : 0ull;
    int c = 0;
    if (mine) {
      const int b0 = s.depth_off[d] - 1, b1 = b0 + s.depth_cnt[d];
      for (int jj = b0 + q; jj < b1; jj += sp) {
        const int j = s.kk[jj];
        const unsigned long long hj = s.nd_pk[2 * j], lj = s.nd_pk[2 * j + 1];
        c += hj < hi || (hj == hi && lj < lo);
      }
    }
    for (int o = sp >> 1; o > 0; o >>= 1) c += __shfl_xor_sync(FULL, c, o);
    if (mine && q == 0) s.nd_slot[node] = (short)(s.depth_off[d] + c);
    __syncthreads();
  } else {
    for (int d = 1; d <= L; ++d) {  // paths too long to pack: one depth at a time
      if (s.depth_cnt[d] == 0) break;  // prefix-closed: deeper levels are empty too
      const bool mine = tid < n_acc && s.nd_depth[tid] == d;
      if (tid < n_acc) {
        const int p = s.nd_parent[tid];
        s.kk[tid] = mine ? (p < 0 ? 0 : s.nd_slot[p]) * k + s.nd_rank[tid] : -1;
      }
      __syncthreads();
      if (mine) {
        const int key = s.kk[tid];
        int c = 0;
        for (int j = 0; j < n_acc; ++j) c += s.kk[j] >= 0 && s.kk[j] < key;
        s.nd_slot[tid] = (short)(s.depth_off[d] + c);
      }
      __syncthreads();
    }
  }
  // ---- outputs
  const int64_t o = (int64_t)b * N;
  const int poff = pos_offset ? pos_offset[b] : 0;
  if (tid == 0) {
    g_tok[o] = anchor_tokens ? anchor_tokens[b] : -1;
    g_par[o] = -1; g_dep[o] = 0; g_rk[o] = -1; g_pos[o] = poff;
    g_sc[o] = 0.f; g_nn[b] = n_acc + 1;
    s.maskrow[0] = 1u;
    if (status) status[b] = s.scalars[4];
  }
  if (tid < n_acc) {
    const int sl = s.nd_slot[tid], p = s.nd_parent[tid], d = s.nd_depth[tid], r = s.nd_rank[tid];
    g_tok[o + sl] = s.tok[(d - 1) * k + r];
    g_par[o + sl] = p < 0 ? 0 : s.nd_slot[p];
    g_dep[o + sl] = d; g_rk[o + sl] = r; g_pos[o + sl] = poff + d;
    g_sc[o + sl] = s.nd_score[tid];
    uint32_t* row = s.maskrow.ptr((long long)sl * mw, mw);
    row[0] |= 1u;  // the root
    for (int a = tid; a >= 0; a = s.nd_parent[a]) {
      const int as = s.nd_slot[a];
      row[as >> 5] |= 1u << (as & 31);
    }
  }
  for (int i = n_acc + 1 + tid; i < N; i += G2_T) {
    g_tok[o + i] = -1; g_par[o + i] = -1; g_dep[o + i] = -1;
    g_rk[o + i] = -1; g_pos[o + i] = -1; g_sc[o + i] = -INFINITY;
  }
  __syncthreads();
  for (int i = tid; i < N * mw; i += G2_T) g_mask[(int64_t)b * N * mw + i] = s.maskrow[i];
}

// Step a3b alone: one CTA per sequence, one thread per slot.
__global__ void __launch_bounds__(G2_T)
k_build_mask(ubt_tree tree, const int32_t* __restrict__ pos_offset) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* rows = reinterpret_cast<uint32_t*>(smem_raw);
  const int b = blockIdx.x, tid = threadIdx.x, N = tree.N, mw = (N + 31) / 32;
  const int64_t o = (int64_t)b * N;
  const int n = tree.n_nodes[b];
  for (int i = tid; i < N * mw; i += G2_T) rows[i] = 0u;
  __syncthreads();
  const int poff = pos_offset ? pos_offset[b] : 0;
  for (int i = tid; i < N; i += G2_T) {
    if (i < n) {
      int a = i;
      for (int step = 0; a >= 0 && step <= N; ++step) {  // bounded: a malformed parent array cannot loop
        rows[(size_t)i * mw + (a >> 5)] |= 1u << (a & 31);
        a = tree.parents[o + a];
      }
      tree.position_ids[o + i] = poff + tree.depths[o + i];
    } else {
      tree.position_ids[o + i] = -1;
    }
  }
  __syncthreads();
  for (int i = tid; i < N * mw; i += G2_T) tree.mask[(int64_t)b * N * mw + i] = rows[i];
}

cudaError_t launch_build_tree(const float* bigram, int B, int L, int k, int N, int W, float zeta,
                              const float* alpha, const float* lambda, const float* anchor_bigram,
                              const int32_t* anchor_tokens, const int32_t* pos_offset,
                              const ubt_tree& out, const MergeParts& parts, int V, int32_t* status, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  TreeLayout lay = tree_layout(L, k, N, W);
  if (lay.total > (size_t)device_info().max_smem_optin) lay = tree_layout(L, k, N);  // without the depth-by-depth arrays
  const size_t smem = lay.total;
  const bool lazy = lay.lazy != 0;
  auto kern = lazy ? k_build_tree<true> : k_build_tree<false>;
  cudaError_t e = lazy ? allow_max_dynamic_smem<k_build_tree<true>>() : allow_max_dynamic_smem<k_build_tree<false>>();
  if (e != cudaSuccess) return e;
  // programmatic launch only when the kernel before it is this library's own streaming kernel
  return launch_kernel(kern, dim3(B), dim3(G2_T), smem, st, parts.part_ms != nullptr, bigram, L, k, N, W,
                       zeta, alpha, lambda, anchor_bigram, anchor_tokens, pos_offset, out, parts, V, status, lay);
}

cudaError_t launch_build_mask(const ubt_tree& tree, const int32_t* pos_offset, cudaStream_t st) {
  if (tree.B == 0) return cudaSuccess;
  const size_t smem = sizeof(uint32_t) * (size_t)tree.N * ((tree.N + 31) / 32);
  k_build_mask<<<tree.B, G2_T, smem, st>>>(tree, pos_offset);
  return cudaGetLastError();
}

#ifdef UBT_BOUNDS_CHECK
// Debug builds only: first out-of-range index seen by the kernels of this file (flag, site, index, limit).
cudaError_t bounds_report_tree(long long out[4]) {
  BoundsReport r;
  cudaError_t e = cudaMemcpyFromSymbol(&r, g_bounds_report, sizeof r);
  out[0] = r.flag; out[1] = r.site; out[2] = r.index; out[3] = r.limit;
  return e;
}
#endif

}  // namespace ubt
