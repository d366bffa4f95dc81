/*
 * CPU oracle for the UBTree draft-tree + verification hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, double-precision
 * statement of what the path computes, written from the paper's definitions.
 * It shares no code, header, table or constant generator with the CUDA
 * library and is never on the product path: only the tests, the smoke check
 * and the benchmark's CPU-baseline leg call it.
 *
 * Every function cites the passage of the paper it follows.  Where the paper
 * is silent the reading taken is stated at the function.
 *
 * Parity pins (tests, no GPU needed): brute-force enumeration of every prefix
 * against eq. 9 directly, tree invariants, closed-form rows (logits = ln of
 * integer weights), numpy / scipy library routines for top-k, log-sum-exp and
 * argmax, the Random123 known-answer vectors for Philox4x32-10, exp() in
 * double for the weight routine, and analytic acceptance statistics.
 *
 * Notation (paper -> here): gamma -> L draft positions, K -> k candidates per
 * position, B (non-root budget) -> N - 1 where N counts tree slots including
 * the root, W -> search width (0 = unbounded), zeta -> depth bonus.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define UBT_ORACLE_F32 0
#define UBT_ORACLE_BF16 1

/* ---------------------------------------------------------------------- */
/* Input widening: bf16 -> double and fp32 -> double are both exact.        */
/* ---------------------------------------------------------------------- */
static float bf16_bits_to_float(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

static float load_f32(const void *base, int dtype, int64_t i) {
  if (dtype == UBT_ORACLE_BF16) return bf16_bits_to_float(((const uint16_t *)base)[i]);
  return ((const float *)base)[i];
}

/* ---------------------------------------------------------------------- */
/* Step 1.  Candidate sets and vocabulary log-softmax.                      */
/*                                                                          */
/* Eq. 3 (Section 3.1.1): q_i = softmax(u_i).  "Candidate Sets": C_i is the */
/* top-K tokens of q_i.  softmax is monotone, so the ranking is taken on    */
/* the raw logits; ties go to the lower token id (reading: paper silent).   */
/* Candidates are ordered best first; the index in that order is the        */
/* candidate's rank r.  cand_lp[r] = u[C_r] - log sum_v exp u[v].           */
/* ---------------------------------------------------------------------- */
int ubt_oracle_topk_logprob(const void *logits, int dtype, int64_t rows, int V, int k,
                            int32_t *cand_ids, double *cand_lp, double *row_lse) {
  if (!logits || rows < 0 || V < 1 || k < 1 || k > V) return 1;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t row = 0; row < rows; ++row) {
    double *x = (double *)malloc(sizeof(double) * (size_t)V);
    char *taken = (char *)calloc((size_t)V, 1);
    if (!x || !taken) { bad = 1; free(x); free(taken); continue; }
    for (int v = 0; v < V; ++v) x[v] = (double)load_f32(logits, dtype, row * (int64_t)V + v);

    /* log-sum-exp over the whole vocabulary (eq. 3 denominator) */
    double m = x[0];
    for (int v = 1; v < V; ++v) if (x[v] > m) m = x[v];
    double sum = 0.0;
    for (int v = 0; v < V; ++v) sum += exp(x[v] - m);
    double lse = m + log(sum);
    if (row_lse) row_lse[row] = lse;

    /* first k under (logit descending, token id ascending): plain selection */
    for (int r = 0; r < k; ++r) {
      int best = -1;
      for (int v = 0; v < V; ++v) {
        if (taken[v]) continue;
        if (best < 0 || x[v] > x[best]) best = v; /* strict >: lower id wins ties */
      }
      taken[best] = 1;
      cand_ids[row * k + r] = best;
      cand_lp[row * k + r] = x[best] - lse;
    }
    free(x);
    free(taken);
  }
  return bad;
}

/* ---------------------------------------------------------------------- */
/* Unigram logits from the proposer state (Section 3.1.1, eq. 3: the logit   */
/* vector of a position is the frozen LM head applied to the position's       */
/* hidden state), followed by the candidate selection above:                  */
/*   u[row][v] = sum_j h[row][j] * W[v][j]      (double; inputs bf16 or fp32) */
/* then the k best under (logit descending, token id ascending) and           */
/*   cand_lp[r] = u[C_r] - log sum_v exp u[v].                                 */
/* W is [V, d] row-major (one row of d weights per token), h is [rows, d].    */
/* row_logits (optional, [rows, V] double) receives u for tests.              */
/* ---------------------------------------------------------------------- */
int ubt_oracle_lm_head_topk(const void *h, const void *W, int dtype, int64_t rows, int d, int V, int k,
                            int32_t *cand_ids, double *cand_lp, double *row_lse, double *row_logits) {
  if (!h || !W || rows < 0 || d < 1 || V < 1 || k < 1 || k > V) return 1;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t row = 0; row < rows; ++row) {
    double *x = (double *)malloc(sizeof(double) * (size_t)V);
    double *hr = (double *)malloc(sizeof(double) * (size_t)d);
    char *taken = (char *)calloc((size_t)V, 1);
    if (!x || !hr || !taken) { bad = 1; free(x); free(hr); free(taken); continue; }
    for (int j = 0; j < d; ++j) hr[j] = (double)load_f32(h, dtype, row * (int64_t)d + j);
    for (int v = 0; v < V; ++v) {
      double acc = 0.0;
      for (int j = 0; j < d; ++j) acc += hr[j] * (double)load_f32(W, dtype, (int64_t)v * d + j);
      x[v] = acc;
    }
    if (row_logits) memcpy(row_logits + row * (int64_t)V, x, sizeof(double) * (size_t)V);
    double m = x[0];
    for (int v = 1; v < V; ++v) if (x[v] > m) m = x[v];
    double sum = 0.0;
    for (int v = 0; v < V; ++v) sum += exp(x[v] - m);
    double lse = m + log(sum);
    if (row_lse) row_lse[row] = lse;
    for (int r = 0; r < k; ++r) {
      int best = -1;
      for (int v = 0; v < V; ++v) {
        if (taken[v]) continue;
        if (best < 0 || x[v] > x[best]) best = v; /* strict >: lower id wins ties */
      }
      taken[best] = 1;
      cand_ids[row * k + r] = best;
      cand_lp[row * k + r] = x[best] - lse;
    }
    free(x); free(hr); free(taken);
  }
  return bad;
}

/* ---------------------------------------------------------------------- */
/* Selector scores (Section 3.1.2, "Parallel Computation", the edge-matrix   */
/* equation; the score of one pair is the low-rank bigram selector of        */
/* Section 2): for predecessor token a and successor token b at position i,  */
/*   delta_i(a, b) = sum_r g_i[r] * phi[a][r] * psi[b][r],                   */
/* g_i = P(h_i) being the projected proposer state of the SUCCESSOR position */
/* and phi, psi the vocabulary-wide codebook tables.  Predecessors are the   */
/* candidates of position i-1; for the first position the only predecessor   */
/* is the anchor token.  Outputs: bigram[b][j][ra][rb] = delta between the   */
/* rank-ra candidate of position j and the rank-rb candidate of position j+1 */
/* (gate of position j+1); anchor_bigram[b][rb] = delta between the anchor   */
/* and the rank-rb candidate of position 0 (gate of position 0).  The sum    */
/* runs over r in index order, in double.                                    */
/* ---------------------------------------------------------------------- */
int ubt_oracle_selector_scores(const void *phi, const void *psi, int dtype, int64_t V, int R, const float *gate,
                               const int32_t *cand_ids, const int32_t *anchor_tokens, int B, int L, int k,
                               double *bigram, double *anchor_bigram) {
  if (!phi || !psi || !gate || !cand_ids || B < 0 || L < 1 || k < 1 || R < 1 || V < 1) return 1;
  if (anchor_bigram && !anchor_tokens) return 1;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int i = 0; i < L; ++i) {
      const float *g = gate + ((int64_t)b * L + i) * R;
      const int npred = i == 0 ? 1 : k;
      if (i == 0 && !anchor_bigram) continue;
      for (int ra = 0; ra < npred; ++ra) {
        const int64_t a = i == 0 ? anchor_tokens[b] : cand_ids[((int64_t)b * L + i - 1) * k + ra];
        for (int rb = 0; rb < k; ++rb) {
          const int64_t t = cand_ids[((int64_t)b * L + i) * k + rb];
          if (a < 0 || a >= V || t < 0 || t >= V) { bad = 1; continue; }
          double sum = 0.0;
          for (int r = 0; r < R; ++r)
            sum += (double)g[r] * (double)load_f32(phi, dtype, a * R + r) * (double)load_f32(psi, dtype, t * R + r);
          if (i == 0) anchor_bigram[(int64_t)b * k + rb] = sum;
          else bigram[(((int64_t)b * (L - 1) + i - 1) * k + ra) * k + rb] = sum;
        }
      }
    }
  }
  return bad;
}

/* ---------------------------------------------------------------------- */
/* Steps 2-3.  Tree construction (Appendix A, Algorithm 1).                 */
/* ---------------------------------------------------------------------- */
typedef struct {
  double score;  /* ell_zeta, eq. 10 */
  int depth;     /* d >= 1 */
  int token;
  int rank;      /* candidate rank of y_d inside C_d */
  int *path;     /* ranks (r_1..r_d); identifies the node (Appendix A, "Path Scores":
                    a node is its complete prefix) */
  int parent;    /* index into the supertree array S, -1 = root */
  int slot;      /* output slot once selected, else -1 */
} onode;

/* Total order Omega, "better first".  For equal scores the paper fixes only
 * that an ancestor goes before its descendants (Appendix A, Global Pruning);
 * an ancestor is always shallower, hence rule 2.  Rules 3-5 are this build's
 * reading that makes the order total: lower token id, lower candidate rank,
 * then the rank path in lexicographic order. */
static int omega_cmp(const void *pa, const void *pb) {
  const onode *a = (const onode *)pa, *b = (const onode *)pb;
  if (a->score > b->score) return -1;
  if (a->score < b->score) return 1;
  if (a->depth != b->depth) return a->depth < b->depth ? -1 : 1;
  if (a->token != b->token) return a->token < b->token ? -1 : 1;
  if (a->rank != b->rank) return a->rank < b->rank ? -1 : 1;
  for (int i = 0; i < a->depth; ++i)
    if (a->path[i] != b->path[i]) return a->path[i] < b->path[i] ? -1 : 1;
  return 0;
}

static double rel_gap(double kept, double dropped) {
  double scale = fabs(kept) > 1.0 ? fabs(kept) : 1.0;
  return (kept - dropped) / scale;
}

/*
 * Inputs per sequence b:
 *   cand_ids[b,L,k], cand_lp[b,L,k]  from step 1
 *   bigram[b,L-1,k,k]   delta_{i+1}(a,b') for a = rank in C_i, b' = rank in C_{i+1}
 *   alpha[L], lambda[L] depth calibration (eq. 5), NULL = 1 (their initial value)
 *   anchor_bigram[b,k]  delta_1(x_t, .) for the anchor -> depth-1 transition, NULL = 0
 *   anchor_tokens[b]    token id stored in the root slot, NULL = -1
 *   pos_offset[b]       position id of the root, NULL = 0
 *   N                   tree slots including the root (the paper's budget B leaves
 *                       the root out, so its B = N - 1; Appendix A, Global Pruning)
 *   W                   search width; 0 = unbounded.  An unbounded or large width
 *                       is run as W_eff = N - 1: every depth of the exact global
 *                       Top-(N-1) holds at most N - 1 nodes and is contained in
 *                       Top_{N-1}(E_d) by induction, so the result is the same.
 *   zeta                depth bonus, <= 0 (eq. 10)
 * Outputs per sequence, slot 0 = root, slots in (depth, parent slot, rank) order,
 * unused slots filled with -1 / -inf / zero mask:
 *   token_ids, parents, depths, cand_rank, position_ids [b,N]; scores [b,N] double;
 *   mask [b,N,mask_words] (bit j of row i set iff j is i or an ancestor of i);
 *   n_nodes[b]; t_out [b,L,k,k] = log q^bi (eq. 9; depth-1 rows use ra = 0 only);
 *   min_cut_gap[b] = smallest relative score gap between the last kept and the
 *   first dropped node over every Top_W / Top_B cut that dropped something
 *   (+inf when nothing was dropped): tells a test whether an fp32
 *   implementation may legitimately pick differently.
 */
int ubt_oracle_build_tree(const int32_t *cand_ids, const double *cand_lp, const float *bigram,
                          int B, int L, int k, int N, int W, double zeta,
                          const float *alpha, const float *lambda, const float *anchor_bigram,
                          const int32_t *anchor_tokens, const int32_t *pos_offset,
                          int32_t *token_ids, int32_t *parents, int32_t *depths,
                          int32_t *cand_rank, int32_t *position_ids, double *scores,
                          uint32_t *mask, int32_t *n_nodes, double *t_out,
                          double *min_cut_gap) {
  if (B < 0 || L < 1 || k < 1 || N < 1 || W < 0 || zeta > 0.0) return 1;
  const int mask_words = (N + 31) / 32;
  const int budget = N - 1;
  int Weff = (W == 0 || W > budget) ? budget : W;
  int bad = 0;

#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    const int32_t *ids = cand_ids + (int64_t)b * L * k;
    const double *lp = cand_lp + (int64_t)b * L * k;
    const float *big = bigram ? bigram + (int64_t)b * (L - 1) * k * k : NULL;
    double *t = (double *)malloc(sizeof(double) * (size_t)L * k * k);
    /* supertree S (union of frontiers) and the extension set E_d */
    size_t capS = (size_t)L * (size_t)(Weff > 0 ? Weff : 1) + 1;
    size_t capE = (size_t)(Weff > 0 ? Weff : 1) * k + (size_t)k;
    onode *S = (onode *)malloc(sizeof(onode) * capS);
    onode *E = (onode *)malloc(sizeof(onode) * capE);
    int *pathpool = (int *)malloc(sizeof(int) * (capS + capE) * (size_t)L);
    if (!t || !S || !E || !pathpool) { bad = 1; free(t); free(S); free(E); free(pathpool); continue; }
    int *Spaths = pathpool, *Epaths = pathpool + capS * (size_t)L;
    double gap = INFINITY;

    /* eq. 5: s_i(a,b') = alpha_i u_i(b') + lambda_i delta_i(a,b').  u_i(b') is
     * taken as the log-probability lp_i(b'); the two differ by a per-position
     * constant that the normalisation of eq. 9 cancels.
     * eq. 9: t_i(a,b') = s_i(a,b') - log sum_{v in C_i} exp s_i(a,v), the
     * normalisation running over the k successor candidates only. */
    for (int i = 0; i < L; ++i) {
      double al = alpha ? (double)alpha[i] : 1.0, la = lambda ? (double)lambda[i] : 1.0;
      int npred = (i == 0) ? 1 : k;
      for (int ra = 0; ra < k; ++ra) {
        double *trow = t + ((size_t)i * k + ra) * k;
        if (ra >= npred) { for (int rb = 0; rb < k; ++rb) trow[rb] = 0.0; continue; }
        double mx = -INFINITY;
        for (int rb = 0; rb < k; ++rb) {
          double delta;
          if (i == 0) delta = anchor_bigram ? (double)anchor_bigram[(int64_t)b * k + rb] : 0.0;
          else delta = (double)big[(((int64_t)(i - 1)) * k + ra) * k + rb];
          trow[rb] = al * lp[i * k + rb] + la * delta;
          if (trow[rb] > mx) mx = trow[rb];
        }
        double sum = 0.0;
        for (int rb = 0; rb < k; ++rb) sum += exp(trow[rb] - mx);
        double lse = mx + log(sum);
        for (int rb = 0; rb < k; ++rb) trow[rb] -= lse;
      }
    }
    if (t_out) memcpy(t_out + (int64_t)b * L * k * k, t, sizeof(double) * (size_t)L * k * k);

    /* depth-wise expansion (eq. 11): the retained set of depth 0 is the root alone, with score 0 */
    int nS = 0;         /* nodes in S */
    int f_lo = -1, f_hi = -1; /* F_{d-1} = S[f_lo..f_hi); (-1,-1) = {root} */
    for (int d = 1; d <= L && Weff > 0; ++d) {
      /* E_d = every retained path extended by every candidate of position d */
      int nE = 0;
      int nparents = (d == 1) ? 1 : (f_hi - f_lo);
      for (int pi = 0; pi < nparents; ++pi) {
        int p = (d == 1) ? -1 : f_lo + pi;
        double pscore = (p < 0) ? 0.0 : S[p].score;
        int prank = (p < 0) ? 0 : S[p].rank;
        for (int r = 0; r < k; ++r) {
          onode *e = &E[nE];
          e->path = Epaths + (size_t)nE * L;
          if (p >= 0) memcpy(e->path, S[p].path, sizeof(int) * (size_t)(d - 1));
          e->path[d - 1] = r;
          /* eq. 9-10: a child adds its pair log-probability and the depth bonus to its parent's score */
          e->score = pscore + t[((size_t)(d - 1) * k + prank) * k + r] + zeta;
          e->depth = d;
          e->rank = r;
          e->token = ids[(d - 1) * k + r];
          e->parent = p;
          e->slot = -1;
          ++nE;
        }
      }
      /* F_d = Top_W(E_d) across all extensions of the depth (eq. 11) */
      qsort(E, (size_t)nE, sizeof(onode), omega_cmp);
      int keep = nE < Weff ? nE : Weff;
      if (nE > keep) {
        double g = rel_gap(E[keep - 1].score, E[keep].score);
        if (g < gap) gap = g;
      }
      f_lo = nS;
      for (int j = 0; j < keep; ++j) {
        S[nS] = E[j];
        S[nS].path = Spaths + (size_t)nS * L;
        memcpy(S[nS].path, E[j].path, sizeof(int) * (size_t)d);
        ++nS;
      }
      f_hi = nS;
    }

    /* T = {root} + Top_B(S) (eq. 12).  Sorting S would lose the parent indices,
     * so sort an index permutation's worth of copies that remember their origin. */
    onode *order = (onode *)malloc(sizeof(onode) * (size_t)(nS > 0 ? nS : 1));
    int *origin = (int *)malloc(sizeof(int) * (size_t)(nS > 0 ? nS : 1));
    if (!order || !origin) { bad = 1; }
    int nsel = 0;
    if (order && origin) {
      for (int j = 0; j < nS; ++j) { order[j] = S[j]; order[j].slot = j; /* origin */ }
      qsort(order, (size_t)nS, sizeof(onode), omega_cmp);
      nsel = nS < budget ? nS : budget;
      if (nS > nsel && nsel > 0) {
        double g = rel_gap(order[nsel - 1].score, order[nsel].score);
        if (g < gap) gap = g;
      }
      for (int j = 0; j < nS; ++j) origin[j] = order[j].slot;
      for (int j = 0; j < nS; ++j) S[j].slot = -1;
      for (int j = 0; j < nsel; ++j) S[origin[j]].slot = -2; /* selected, slot pending */
      /* the selection must be prefix-closed (Appendix A, Global Pruning) */
      for (int j = 0; j < nS; ++j)
        if (S[j].slot == -2 && S[j].parent >= 0 && S[S[j].parent].slot == -1) bad = 1;
    }

    /* Emission order (reading: paper silent).  Slot 0 is the root; the rest go
     * depth by depth, inside a depth by (parent slot, candidate rank). */
    int32_t *tok = token_ids + (int64_t)b * N, *par = parents + (int64_t)b * N;
    int32_t *dep = depths + (int64_t)b * N, *rk = cand_rank + (int64_t)b * N;
    int32_t *pos = position_ids + (int64_t)b * N;
    double *sc = scores + (int64_t)b * N;
    uint32_t *mk = mask + (int64_t)b * N * mask_words;
    for (int i = 0; i < N; ++i) {
      tok[i] = par[i] = dep[i] = rk[i] = pos[i] = -1;
      sc[i] = -INFINITY;
    }
    memset(mk, 0, sizeof(uint32_t) * (size_t)N * mask_words);
    int off = pos_offset ? pos_offset[b] : 0;
    tok[0] = anchor_tokens ? anchor_tokens[b] : -1;
    par[0] = -1; dep[0] = 0; rk[0] = -1; pos[0] = off; sc[0] = 0.0;
    int next = 1;
    for (int d = 1; d <= L; ++d) {
      /* repeatedly take the not-yet-placed selected node of depth d with the
       * smallest (parent slot, rank) */
      for (;;) {
        int best = -1;
        for (int j = 0; j < nS; ++j) {
          if (S[j].slot != -2 || S[j].depth != d) continue;
          if (best < 0) { best = j; continue; }
          int pj = S[j].parent < 0 ? 0 : S[S[j].parent].slot;
          int pb = S[best].parent < 0 ? 0 : S[S[best].parent].slot;
          if (pj < pb || (pj == pb && S[j].rank < S[best].rank)) best = j;
        }
        if (best < 0) break;
        int i = next++;
        S[best].slot = i;
        tok[i] = S[best].token;
        par[i] = S[best].parent < 0 ? 0 : S[S[best].parent].slot;
        dep[i] = d;
        rk[i] = S[best].rank;
        pos[i] = off + d;
        sc[i] = S[best].score;
      }
    }
    n_nodes[b] = next;
    /* ancestor-closure mask: row 0 = {0}; row i = row parent(i) + bit i */
    mk[0] = 1u;
    for (int i = 1; i < next; ++i) {
      memcpy(mk + (size_t)i * mask_words, mk + (size_t)par[i] * mask_words,
             sizeof(uint32_t) * (size_t)mask_words);
      mk[(size_t)i * mask_words + (i >> 5)] |= 1u << (i & 31);
    }
    if (min_cut_gap) min_cut_gap[b] = gap;
    free(order); free(origin);
    free(t); free(S); free(E); free(pathpool);
  }
  return bad;
}

/* ---------------------------------------------------------------------- */
/* Step 4.  Verification (Appendix A, "Verification via Tree-attention").   */
/* ---------------------------------------------------------------------- */

/* Greedy pick (T_infer = 0): the row maximum; ties to the lower token id
 * (reading: paper silent). */
static int32_t greedy_pick(const void *z, int dtype, int64_t row, int V) {
  int best = 0;
  double bv = (double)load_f32(z, dtype, row * (int64_t)V);
  for (int v = 1; v < V; ++v) {
    double x = (double)load_f32(z, dtype, row * (int64_t)V + v);
    if (x > bv) { bv = x; best = v; }
  }
  return best;
}

/* Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3"). */
void ubt_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * Sampling weights (T_infer > 0).  The paper says only that the walk follows
 * what the target model samples at each node (Appendix A, verification); this
 * build's reading pins the sampler so
 * that a pick is a pure function of (row, temperature, seed, b, n):
 *
 *   m  = max_v z[v]                          (fp32, exact)
 *   a  = fl32(log2(e) / T)   as fl32(0x1.715476p+0f * fl32(1/T))
 *   c  = -fl32(m * a)
 *   y  = max(fma(z[v], a, c), -42)           (one rounding; y <= ~0)
 *   n  = nearest integer to y (ties to even, via +/- 1.5*2^23), f = y - n
 *   p  = 1 + f(c1 + f(c2 + f(c3 + f(c4 + f c5))))   fma Horner, ~2^f, rel. err 1.6e-7
 *   w  = trunc(p * 2^(n+40))                 unsigned 64-bit integer
 *
 * The weights are integers, so their sum and every prefix sum are independent
 * of the order of addition.  One Philox4x32-10 draw per node, key = (seed low,
 * seed high), counter = (n, b, 0, 0): R = x0 | x1 << 32, theta = floor(R *
 * total / 2^64), pick = the smallest v whose inclusive prefix sum exceeds theta.
 * Every step is a single IEEE operation, hence bit-reproducible.
 */
static const float EXP2_C1 = 0x1.62e42cp-1f, EXP2_C2 = 0x1.ebf9bcp-3f, EXP2_C3 = 0x1.c6b54ap-5f,
                   EXP2_C4 = 0x1.3cea8p-7f, EXP2_C5 = 0x1.5c7746p-10f;

uint64_t ubt_oracle_weight(float z, float a, float c) {
  float y = fmaf(z, a, c);
  if (y < -42.0f) y = -42.0f;
  float big = 12582912.0f; /* 1.5 * 2^23 */
  float tmp = y + big;
  float nf = tmp - big;
  float f = y - nf;
  float p = EXP2_C5;
  p = fmaf(p, f, EXP2_C4);
  p = fmaf(p, f, EXP2_C3);
  p = fmaf(p, f, EXP2_C2);
  p = fmaf(p, f, EXP2_C1);
  p = fmaf(p, f, 1.0f);
  float e = ldexpf(p, (int)nf + 40); /* exact power-of-two scaling */
  return (uint64_t)e;                /* truncation; e >= 0 */
}

void ubt_oracle_weight_consts(float row_max, float temperature, float *a, float *c) {
  float inv_t = 1.0f / temperature;
  *a = 0x1.715476p+0f * inv_t;
  *c = -(row_max * *a);
}

/* Inclusive prefix sums of the integer weights of one row; returns the total. */
uint64_t ubt_oracle_row_cdf(const void *z, int dtype, int64_t row, int V, float temperature,
                            uint64_t *prefix /* [V] or NULL */) {
  float m = load_f32(z, dtype, row * (int64_t)V);
  for (int v = 1; v < V; ++v) {
    float x = load_f32(z, dtype, row * (int64_t)V + v);
    if (x > m) m = x;
  }
  float a, c;
  ubt_oracle_weight_consts(m, temperature, &a, &c);
  uint64_t acc = 0;
  for (int v = 0; v < V; ++v) {
    acc += ubt_oracle_weight(load_f32(z, dtype, row * (int64_t)V + v), a, c);
    if (prefix) prefix[v] = acc;
  }
  return acc;
}

uint64_t ubt_oracle_threshold(uint64_t seed, uint32_t b, uint32_t n, uint64_t total) {
  uint32_t ctr[4] = {n, b, 0u, 0u}, key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)}, x[4];
  ubt_oracle_philox4x32_10(ctr, key, x);
  uint64_t r = (uint64_t)x[0] | ((uint64_t)x[1] << 32);
  return (uint64_t)(((unsigned __int128)r * (unsigned __int128)total) >> 64);
}

static int32_t sample_pick(const void *z, int dtype, int64_t row, int V, float temperature,
                           uint64_t seed, uint32_t b, uint32_t n) {
  uint64_t total = ubt_oracle_row_cdf(z, dtype, row, V, temperature, NULL);
  uint64_t theta = ubt_oracle_threshold(seed, b, n, total);
  float m = load_f32(z, dtype, row * (int64_t)V);
  for (int v = 1; v < V; ++v) {
    float x = load_f32(z, dtype, row * (int64_t)V + v);
    if (x > m) m = x;
  }
  float a, c;
  ubt_oracle_weight_consts(m, temperature, &a, &c);
  uint64_t acc = 0;
  for (int v = 0; v < V; ++v) {
    acc += ubt_oracle_weight(load_f32(z, dtype, row * (int64_t)V + v), a, c);
    if (acc > theta) return v;
  }
  return V - 1; /* unreachable: theta < total */
}

/*
 * The walk.  From the root, take the target's pick x at the current node; if a
 * child of the current node carries token x, move to it and count it accepted;
 * otherwise x is the bonus token and the walk ends (Appendix A, verification:
 * the walk stops at the first pick that no child carries and keeps that pick as
 * the bonus token).  Siblings carry distinct
 * tokens, so the child is unique.  accepted_len counts draft tokens only; the
 * paper's tau (Section 2) is accepted_len + 1.
 *
 * mode 0 = greedy, 1 = sampling.  node_pick (optional, [B,N]) receives the pick
 * of EVERY row, used or not; without it only the visited rows are evaluated.
 * accepted_nodes / out_tokens are [B,L+1], padded with -1.
 */
int ubt_oracle_verify(const int32_t *token_ids, const int32_t *parents, const int32_t *n_nodes,
                      int B, int N, int L, const void *target_logits, int dtype, int V, int mode,
                      uint64_t seed, float temperature, int32_t *accepted_len,
                      int32_t *accepted_nodes, int32_t *out_tokens, int32_t *bonus_token,
                      int32_t *node_pick) {
  if (B < 0 || N < 1 || L < 1 || V < 1 || (mode != 0 && mode != 1)) return 1;
  if (mode == 1 && !(temperature > 0.0f)) return 1;
  if (node_pick) {
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t row = 0; row < (int64_t)B * N; ++row) {
      uint32_t b = (uint32_t)(row / N), n = (uint32_t)(row % N);
      node_pick[row] = mode == 0 ? greedy_pick(target_logits, dtype, row, V)
                                 : sample_pick(target_logits, dtype, row, V, temperature, seed, b, n);
    }
  }
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    const int32_t *tok = token_ids + (int64_t)b * N, *par = parents + (int64_t)b * N;
    int32_t *an = accepted_nodes + (int64_t)b * (L + 1), *ot = out_tokens + (int64_t)b * (L + 1);
    for (int j = 0; j <= L; ++j) an[j] = ot[j] = -1;
    int cur = 0, acc = 0;
    an[0] = 0;
    for (;;) {
      int64_t row = (int64_t)b * N + cur;
      int32_t x = node_pick ? node_pick[row]
                 : mode == 0 ? greedy_pick(target_logits, dtype, row, V)
                             : sample_pick(target_logits, dtype, row, V, temperature, seed,
                                           (uint32_t)b, (uint32_t)cur);
      int child = -1;
      for (int c = 1; c < n_nodes[b]; ++c)
        if (par[c] == cur && tok[c] == x) { child = c; break; }
      if (child < 0) { bonus_token[b] = x; ot[acc] = x; break; }
      ot[acc] = x;
      ++acc;
      an[acc] = child;
      cur = child;
    }
    accepted_len[b] = acc;
  }
  return 0;
}

/*
 * The walk alone, for picks that come from elsewhere (Appendix A, verification): from the root, move to the child
 * that carries the pick of the current slot; the first pick that no child carries ends the walk and is the bonus
 * token.  picks[B,N] holds the target's token at every slot; only the slots the walk visits are read.  Outputs as
 * ubt_oracle_verify.
 */
int ubt_oracle_walk_picks(const int32_t *token_ids, const int32_t *parents, const int32_t *n_nodes,
                          int B, int N, int L, const int32_t *picks, int32_t *accepted_len,
                          int32_t *accepted_nodes, int32_t *out_tokens, int32_t *bonus_token) {
  if (B < 0 || N < 1 || L < 1) return 1;
  for (int b = 0; b < B; ++b) {
    const int32_t *tok = token_ids + (int64_t)b * N, *par = parents + (int64_t)b * N;
    int32_t *an = accepted_nodes + (int64_t)b * (L + 1), *ot = out_tokens + (int64_t)b * (L + 1);
    for (int j = 0; j <= L; ++j) an[j] = ot[j] = -1;
    int cur = 0, acc = 0;
    an[0] = 0;
    for (;;) {
      const int32_t x = picks[(int64_t)b * N + cur];
      ot[acc] = x;
      int child = -1;
      for (int c = 1; c < n_nodes[b]; ++c)
        if (par[c] == cur && tok[c] == x) { child = c; break; }
      if (child < 0) { bonus_token[b] = x; break; }
      ++acc;
      an[acc] = child;
      cur = child;
    }
    accepted_len[b] = acc;
  }
  return 0;
}

/*
 * Many sampling walks over one sequence's tree from precomputed row CDFs
 * (cdf[n] = inclusive prefix sums of row n, as ubt_oracle_row_cdf writes them).
 * Same definition as above with the prefix sums looked up instead of summed
 * again; used for acceptance statistics over many seeds.
 */
int ubt_oracle_walks_from_cdf(const int32_t *token_ids, const int32_t *parents, int n_nodes,
                              int V, const uint64_t *cdf /* [N,V] */, uint32_t b,
                              const uint64_t *seeds, int n_seeds, int32_t *accepted_len,
                              int32_t *bonus_token) {
  for (int s = 0; s < n_seeds; ++s) {
    int cur = 0, acc = 0;
    for (;;) {
      const uint64_t *p = cdf + (int64_t)cur * V;
      uint64_t theta = ubt_oracle_threshold(seeds[s], b, (uint32_t)cur, p[V - 1]);
      int lo = 0, hi = V - 1; /* smallest v with p[v] > theta */
      while (lo < hi) {
        int mid = lo + (hi - lo) / 2;
        if (p[mid] > theta) hi = mid; else lo = mid + 1;
      }
      int child = -1;
      for (int c = 1; c < n_nodes; ++c)
        if (parents[c] == cur && token_ids[c] == lo) { child = c; break; }
      if (child < 0) { bonus_token[s] = lo; break; }
      ++acc;
      cur = child;
    }
    accepted_len[s] = acc;
  }
  return 0;
}

int ubt_oracle_num_threads(void) {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
#endif
  return n;
}
