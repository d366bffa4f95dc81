// Steps a2, a3, a3b: candidate-pair log-probabilities, budgeted tree expansion, tree-attention inputs.
//
// One CTA per sequence.  The pair table t[i][ra][rb] = log q^bi (eq. 5 + eq. 9) lives in shared
// memory with, for every (i, ra), the successors sorted best first.  Algorithm 1 is run as a
// best-first search: the frontier holds, per expanded node, its best not-yet-taken child; a pop
// takes the best frontier entry under the total order (score desc, depth asc, token asc, rank path
// asc), replaces it by its next sibling and adds its own first child.  Because every pair
// log-probability is <= 0 and zeta <= 0, scores never increase along a path, so pops come out in
// the global order; a node popped when its depth already holds W nodes is outside Top_W(E_d) and is
// dropped with its later siblings.  N-1 accepted pops give Top_B of the supertree (eq. 11-12).
#include "ubt_internal.h"

namespace ubt {

constexpr int G2_T = 256;

struct TreeSmem {
  Span<float> t;            // [L,k,k]
  Span<unsigned char> ord;  // [L,k,k]  successor ranks sorted by (t desc, token asc)
  Span<float> lp;           // [L,k]
  Span<int> tok;            // [L,k]
  Span<uint32_t> f_key;     // frontier, <= N entries
  Span<float> f_score;
  Span<short> f_parent;     // accepted-node index of the parent, -1 = root
  Span<unsigned char> f_sib;  // position in the parent's sorted successor list
  Span<short> nd_parent;    // accepted nodes in pop order, <= N-1
  Span<unsigned char> nd_depth;
  Span<unsigned char> nd_rank;
  Span<float> nd_score;
  Span<short> nd_slot;
  Span<short> bkt;          // nodes grouped by depth
  Span<int> kk;             // per-depth sort keys
  Span<int> depth_cnt;      // [L+2]
  Span<int> depth_off;      // [L+2]
  Span<uint32_t> maskrow;   // [N, mask_words]
  Span<int> scalars;        // [0] = accepted count
};

__host__ __device__ inline size_t tree_carve(TreeSmem* s, unsigned char* base, int L, int k, int N) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t at = off;
    off = (off + bytes + 15) / 16 * 16;
    return at;
  };
  const int mw = (N + 31) / 32;
  const long long lkk = (long long)L * k * k, lk = (long long)L * k;
  size_t o_t = take(sizeof(float) * lkk), o_ord = take((size_t)lkk);
  size_t o_lp = take(sizeof(float) * lk), o_tok = take(sizeof(int) * lk);
  size_t o_fk = take(sizeof(uint32_t) * (N + 1)), o_fs = take(sizeof(float) * (N + 1));
  size_t o_fp = take(sizeof(short) * (N + 1)), o_fb = take(N + 1);
  size_t o_np = take(sizeof(short) * N), o_nd = take(N), o_nr = take(N);
  size_t o_ns = take(sizeof(float) * N), o_nl = take(sizeof(short) * N), o_bk = take(sizeof(short) * N);
  size_t o_kk = take(sizeof(int) * N);
  size_t o_dc = take(sizeof(int) * (L + 2)), o_do = take(sizeof(int) * (L + 2));
  size_t o_mk = take(sizeof(uint32_t) * N * mw), o_sc = take(sizeof(int) * 4);
  if (s) {
    s->t = Span<float>((float*)(base + o_t), lkk, 101);
    s->ord = Span<unsigned char>(base + o_ord, lkk, 102);
    s->lp = Span<float>((float*)(base + o_lp), lk, 103);
    s->tok = Span<int>((int*)(base + o_tok), lk, 104);
    s->f_key = Span<uint32_t>((uint32_t*)(base + o_fk), N + 1, 105);
    s->f_score = Span<float>((float*)(base + o_fs), N + 1, 106);
    s->f_parent = Span<short>((short*)(base + o_fp), N + 1, 107);
    s->f_sib = Span<unsigned char>(base + o_fb, N + 1, 108);
    s->nd_parent = Span<short>((short*)(base + o_np), N, 109);
    s->nd_depth = Span<unsigned char>(base + o_nd, N, 110);
    s->nd_rank = Span<unsigned char>(base + o_nr, N, 111);
    s->nd_score = Span<float>((float*)(base + o_ns), N, 112);
    s->nd_slot = Span<short>((short*)(base + o_nl), N, 113);
    s->bkt = Span<short>((short*)(base + o_bk), N, 114);
    s->kk = Span<int>((int*)(base + o_kk), N, 115);
    s->depth_cnt = Span<int>((int*)(base + o_dc), L + 2, 116);
    s->depth_off = Span<int>((int*)(base + o_do), L + 2, 117);
    s->maskrow = Span<uint32_t>((uint32_t*)(base + o_mk), (long long)N * mw, 118);
    s->scalars = Span<int>((int*)(base + o_sc), 4, 119);
  }
  return off;
}

size_t tree_smem_bytes(int L, int k, int N) { return tree_carve(nullptr, nullptr, L, k, N); }

__global__ void __launch_bounds__(G2_T)
k_build_tree(const float* __restrict__ bigram, int L, int k, int N, int W, float zeta,
             const float* __restrict__ alpha, const float* __restrict__ lambda,
             const float* __restrict__ anchor_bigram, const int32_t* __restrict__ anchor_tokens,
             const int32_t* __restrict__ pos_offset, ubt_tree out) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TreeSmem s;
  tree_carve(&s, smem_raw, L, k, N);
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const int kk2 = k * k, mw = (N + 31) / 32, budget = N - 1;
  const long long nB = gridDim.x;
  const Span<const float> g_lp(out.cand_logprob, nB * L * k, 201), g_big(bigram, nB * (L - 1) * kk2, 203);
  const Span<const int32_t> g_ids(out.cand_ids, nB * L * k, 202);
  const Span<int32_t> g_tok(out.token_ids, nB * N, 211), g_par(out.parents, nB * N, 212), g_dep(out.depths, nB * N, 213);
  const Span<int32_t> g_rk(out.cand_rank, nB * N, 214), g_pos(out.position_ids, nB * N, 215), g_nn(out.n_nodes, nB, 216);
  const Span<float> g_sc(out.scores, nB * N, 217);
  const Span<uint32_t> g_mask(out.mask, nB * N * mw, 218);

  // ---- stage candidates and raw selector scores
  for (int i = tid; i < L * k; i += G2_T) {
    s.lp[i] = g_lp[(int64_t)b * L * k + i];
    s.tok[i] = g_ids[(int64_t)b * L * k + i];
  }
  for (int i = tid; i < L * kk2; i += G2_T) {
    float d = 0.f;
    if (i < kk2) {
      if (i < k && anchor_bigram) d = anchor_bigram[(int64_t)b * k + i];  // only predecessor row 0 exists
    } else {
      d = g_big[(int64_t)b * (L - 1) * kk2 + (i - kk2)];
    }
    s.t[i] = d;
  }
  for (int i = tid; i < L + 2; i += G2_T) s.depth_cnt[i] = 0;
  for (int i = tid; i < N * mw; i += G2_T) s.maskrow[i] = 0u;
  __syncthreads();

  // ---- eq. 5 and eq. 9: one thread per (position, predecessor) row
  const int nrows = 1 + (L - 1) * k;
  for (int r = tid; r < nrows; r += G2_T) {
    const int i = r == 0 ? 0 : 1 + (r - 1) / k;
    const int ra = r == 0 ? 0 : (r - 1) % k;
    float* row = s.t.ptr(((long long)i * k + ra) * k, k);
    const float al = alpha ? alpha[i] : 1.f, la = lambda ? lambda[i] : 1.f;
    float mx = -INFINITY;
    for (int rb = 0; rb < k; ++rb) {
      float v = al * s.lp[i * k + rb] + la * row[rb];
      row[rb] = v;
      mx = fmaxf(mx, v);
    }
    float sum = 0.f;
    for (int rb = 0; rb < k; ++rb) sum += expf(row[rb] - mx);
    const float lse = mx + logf(sum);
    for (int rb = 0; rb < k; ++rb) row[rb] -= lse;
  }
  __syncthreads();
  // successors of every row sorted by (t desc, token asc)
  for (int q = tid; q < nrows * k; q += G2_T) {
    const int r = q / k, rb = q - r * k;
    const int i = r == 0 ? 0 : 1 + (r - 1) / k;
    const int ra = r == 0 ? 0 : (r - 1) % k;
    const float* row = s.t.ptr(((long long)i * k + ra) * k, k);
    const int* tk = s.tok.ptr((long long)i * k, k);
    // integer keys and a final index tie-break keep this a permutation whatever the values are (even NaN)
    const uint32_t kv = f2key(row[rb]);
    int rank = 0;
    for (int j = 0; j < k; ++j) {
      const uint32_t kj = f2key(row[j]);
      rank += (kj > kv) || (kj == kv && (tk[j] < tk[rb] || (tk[j] == tk[rb] && j < rb)));
    }
    s.ord[((size_t)i * k + ra) * k + rank] = (unsigned char)rb;
  }
  __syncthreads();

  // ---- best-first expansion (warp 0)
  if (tid < 32) {
    int f_cnt = 0, n_acc = 0;
    if (budget > 0) {
      const int r0 = s.ord[0];
      const float sc = s.t[r0] + zeta;
      if (lane == 0) {
        s.f_key[0] = f2key(sc); s.f_score[0] = sc; s.f_parent[0] = -1; s.f_sib[0] = 0;
      }
      f_cnt = 1;
    }
    __syncwarp();
    while (n_acc < budget) {
      uint32_t bk = 0; int bi = -1; bool dup = false;
      for (int i = lane; i < f_cnt; i += 32) {
        const uint32_t key = s.f_key[i];
        if (key > bk) { bk = key; bi = i; dup = false; }
        else if (key == bk && key != 0) dup = true;
      }
      const uint32_t maxk = __reduce_max_sync(FULL, bk);
      if (maxk == 0) break;  // frontier exhausted
      const unsigned holders = __ballot_sync(FULL, bk == maxk);
      const bool tie = __any_sync(FULL, bk == maxk && dup) || __popc(holders) > 1;
      int wi;
      if (!tie) {
        wi = __shfl_sync(FULL, bi, __ffs(holders) - 1);
      } else {
        int best = -1;
        if (lane == 0) {  // exact ties: depth asc, token asc, then rank path lexicographic
          int bd = 0, bt = 0;
          for (int i = 0; i < f_cnt; ++i) {
            if (s.f_key[i] != maxk) continue;
            const int p = s.f_parent[i];
            const int d = p < 0 ? 1 : s.nd_depth[p] + 1;
            const int pr = p < 0 ? 0 : s.nd_rank[p];
            const int tkn = s.tok[(d - 1) * k + s.ord[((size_t)(d - 1) * k + pr) * k + s.f_sib[i]]];
            bool better;
            if (best < 0) better = true;
            else if (d != bd) better = d < bd;
            else if (tkn != bt) better = tkn < bt;
            else {
              int pa = p, pb = s.f_parent[best], ra = 0, rb = 0;
              while (pa != pb) {
                ra = s.nd_rank[pa]; rb = s.nd_rank[pb];
                pa = s.nd_parent[pa]; pb = s.nd_parent[pb];
              }
              better = ra < rb;
            }
            if (better) { best = i; bd = d; bt = tkn; }
          }
        }
        wi = __shfl_sync(FULL, best, 0);
      }
      const int p = s.f_parent[wi], j = s.f_sib[wi];
      const int d = p < 0 ? 1 : s.nd_depth[p] + 1;
      const int pr = p < 0 ? 0 : s.nd_rank[p];
      const float score = s.f_score[wi];
      const int r = s.ord[((size_t)(d - 1) * k + pr) * k + j];
      const int dc = s.depth_cnt[d];
      __syncwarp();
      if (W > 0 && dc >= W) {  // outside Top_W(E_d); so are its later siblings
        if (lane == 0) s.f_key[wi] = 0u;
        __syncwarp();
        continue;
      }
      const int n = n_acc++;
      if (lane == 0) {
        s.nd_parent[n] = (short)p; s.nd_depth[n] = (unsigned char)d; s.nd_rank[n] = (unsigned char)r;
        s.nd_score[n] = score;
        s.bkt[n] = (short)dc;  // position inside its depth, in pop order (re-bucketed below)
        s.depth_cnt[d] = dc + 1;
        if (j + 1 < k) {
          const int r2 = s.ord[((size_t)(d - 1) * k + pr) * k + j + 1];
          const float ps = p < 0 ? 0.f : s.nd_score[p];
          const float s2 = ps + s.t[((size_t)(d - 1) * k + pr) * k + r2] + zeta;
          s.f_score[wi] = s2; s.f_key[wi] = f2key(s2); s.f_sib[wi] = (unsigned char)(j + 1);
        } else {
          s.f_key[wi] = 0u;
        }
        if (d < L) {
          const int r3 = s.ord[((size_t)d * k + r) * k];
          const float s3 = score + s.t[((size_t)d * k + r) * k + r3] + zeta;
          s.f_score[f_cnt] = s3; s.f_key[f_cnt] = f2key(s3);
          s.f_parent[f_cnt] = (short)n; s.f_sib[f_cnt] = 0;
        }
      }
      if (d < L) ++f_cnt;
      __syncwarp();
    }
    if (lane == 0) s.scalars[0] = n_acc;
  }
  __syncthreads();

  // ---- canonical slots: root 0, then depth by depth ordered by (parent slot, rank)
  const int n_acc = s.scalars[0];
  if (tid == 0) {
    int off = 1;
    for (int d = 1; d <= L; ++d) { s.depth_off[d] = off; off += s.depth_cnt[d]; }
  }
  __syncthreads();
  short mynode_dpos = -1;
  if (tid < n_acc) mynode_dpos = s.bkt[tid];
  __syncthreads();
  if (tid < n_acc) s.bkt[s.depth_off[s.nd_depth[tid]] - 1 + mynode_dpos] = (short)tid;
  __syncthreads();
  for (int d = 1; d <= L; ++d) {
    const int cnt = s.depth_cnt[d];
    if (cnt == 0) break;  // prefix-closed: deeper levels are empty too
    const int off = s.depth_off[d];
    int node = -1, key = 0;
    if (tid < cnt) {
      node = s.bkt[off - 1 + tid];
      const int p = s.nd_parent[node];
      key = (p < 0 ? 0 : s.nd_slot[p]) * k + s.nd_rank[node];
      s.kk[tid] = key;
    }
    __syncthreads();
    if (tid < cnt) {
      int c = 0;
      for (int j = 0; j < cnt; ++j) c += s.kk[j] < key;
      s.nd_slot[node] = (short)(off + c);
    }
    __syncthreads();
  }

  // ---- outputs
  const int64_t o = (int64_t)b * N;
  const int poff = pos_offset ? pos_offset[b] : 0;
  if (tid == 0) {
    g_tok[o] = anchor_tokens ? anchor_tokens[b] : -1;
    g_par[o] = -1; g_dep[o] = 0; g_rk[o] = -1; g_pos[o] = poff;
    g_sc[o] = 0.f; g_nn[b] = n_acc + 1;
    s.maskrow[0] = 1u;
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
                              const ubt_tree& out, cudaStream_t st) {
  if (B == 0) return cudaSuccess;
  const size_t smem = tree_smem_bytes(L, k, N);
  cudaError_t e = cudaFuncSetAttribute(k_build_tree, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  k_build_tree<<<B, G2_T, smem, st>>>(bigram, L, k, N, W, zeta, alpha, lambda, anchor_bigram,
                                      anchor_tokens, pos_offset, out);
  return cudaGetLastError();
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
