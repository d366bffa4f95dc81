/*
 * ubt.h -- C ABI of the UBTree draft-tree + verification hot path on NVIDIA B200 (sm_100a).
 *
 * The library computes, for a batch of B independent sequences:
 *   a1  per-position vocabulary log-softmax and top-k candidates          (paper eq. 3, "Candidate Sets")
 *   a2  combine with bigram transition scores, normalise over candidates  (eq. 5, eq. 9)
 *   a3  best-path expansion into a node-budgeted draft tree               (eq. 10-12, Algorithm 1)
 *   a3b tree-attention inputs: position ids and packed ancestor bitmask   (Section 3.1.3, Appendix A)
 *   a4  acceptance walk against target logits, plus the bonus token       (Appendix A, verification)
 *
 * Conventions that hold for every entry point unless it says otherwise
 *   - Pointers named in a struct or argument list are DEVICE pointers owned by the caller; the
 *     library never allocates, frees or synchronises.  All work is enqueued on `cuda_stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream) and keeps stream order: no
 *     input is read, and no output or workspace written, before the work in front of the call on
 *     that stream has completed, and work enqueued behind the call sees all of its results.  The one
 *     exception is opt-in (ubt_verify_opts.early_start).
 *   - Tensors are dense, row-major, in the shapes given; base pointers must be 16-byte aligned.
 *   - Inputs are read-only.  Outputs and the workspace are overwritten; workspace content on entry
 *     is irrelevant.
 *   - Argument errors are detected on the host and returned before anything is launched.
 *     A failed launch returns UBT_ERR_CUDA.  Nothing in the library traps; the only device-side waits
 *     (for a bulk copy to land) are bounded and counted by ubt_debug_ring_timeouts().
 *   - Logits must be free of NaN and +inf (-inf is allowed; each row must hold at least k entries
 *     greater than -inf).  Nothing traps on a violation and every result stays memory-safe, but the
 *     results of the sequence concerned are unspecified.  The calls detect it at no extra pass: pass a
 *     `status` array in the options to learn which sequences were affected.
 *
 * Sizes: B sequences, L draft positions (the paper's gamma), V vocabulary, k candidates per position
 * (the paper's K), N = node budget = tree slots INCLUDING the root (the paper's budget B counts
 * non-root nodes only, so its B equals N - 1).
 * Limits (else UBT_ERR_UNSUPPORTED): 1 <= k <= 64, k <= V < 2^31, 1 <= N <= 256, 1 <= L <= 64.
 * While the per-sequence pair table (L*k*k*5 bytes) fits in 160 KiB of shared memory all its rows are
 * prepared in parallel; larger shapes (the paper's K = 64 with 15 positions is one) are served from a
 * cache of the rows the search touches, each prepared when first needed -- same result, more latency.
 */
#ifndef UBT_H_
#define UBT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  UBT_OK = 0,
  UBT_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, size out of range, k > V, zeta > 0 ... */
  UBT_ERR_UNSUPPORTED = 2, /* valid request beyond the compiled limits above */
  UBT_ERR_WORKSPACE = 3,   /* workspace NULL or smaller than ubt_*_workspace_bytes() */
  UBT_ERR_CUDA = 4,        /* a CUDA call or kernel launch failed */
  UBT_ERR_STATIC_SCRATCH = 5, /* request larger than the built-in scratch of ubt_verify_tree_static */
  UBT_ERR_NONFINITE = 6    /* host-buffer forms with validate_finite: a NaN or +inf among the logits */
} ubt_status;

/* Bits of the per-sequence status words (ubt_draft_opts.status, ubt_verify_opts.status). */
#define UBT_STATUS_NONFINITE 1    /* a NaN or +inf among the sequence's logits: its results are unspecified */
#define UBT_STATUS_WAIT_GAVE_UP 2 /* a bounded device-side wait gave up: its results are undefined */

typedef enum { UBT_F32 = 0, UBT_BF16 = 1 } ubt_dtype;
typedef enum { UBT_VERIFY_GREEDY = 0, UBT_VERIFY_SAMPLE = 1 } ubt_verify_mode;

/*
 * A batch of draft trees.  Slot 0 of every sequence is the root (the empty draft prefix; Appendix A,
 * "Path Scores").  Slots 1..n_nodes-1 hold the selected nodes ordered by (depth, parent slot,
 * candidate rank), so parents[i] < i and the children of one parent are contiguous.  Unused slots
 * n_nodes..N-1 hold -1 (scores: -inf; mask rows: zero).
 */
typedef struct ubt_tree {
  int32_t B, N, L, k, mask_words; /* mask_words = ceil(N / 32) */
  int32_t *token_ids;             /* [B,N]  token of the node; root: anchor token or -1 */
  int32_t *parents;               /* [B,N]  slot of the parent; root: -1 */
  int32_t *depths;                /* [B,N]  root: 0 */
  int32_t *position_ids;          /* [B,N]  pos_offset[b] + depth */
  int32_t *cand_rank;             /* [B,N]  rank of the node's token inside its position's candidates */
  float *scores;                  /* [B,N]  cumulative log-probability ell_zeta (eq. 9-10); root: 0 */
  uint32_t *mask;                 /* [B,N,mask_words]  bit j of row i (word j>>5, bit j&31) set iff
                                     slot j is slot i or an ancestor of it */
  int32_t *n_nodes;               /* [B]    used slots, root included */
  int32_t *cand_ids;              /* [B,L,k] candidate token ids, best first (logit desc, id asc) */
  float *cand_logprob;            /* [B,L,k] their vocabulary log-softmax values */
} ubt_tree;

/* Options of the tree construction; pass NULL for the defaults written beside each field. */
typedef struct ubt_draft_opts {
  int32_t search_width;         /* W of eq. 11; 0 = unbounded (default).  The paper runs W = 12. */
  float depth_bonus;            /* zeta of eq. 10, must be <= 0; default 0 */
  const float *alpha;           /* [L] depth calibration of eq. 5; NULL = 1 */
  const float *lambda;          /* [L] depth calibration of eq. 5; NULL = 1 */
  const float *anchor_bigram;   /* [B,k] selector score of the anchor -> depth-1 transition; NULL = 0 */
  const int32_t *anchor_tokens; /* [B] token stored in the root slot; NULL = -1 */
  const int32_t *pos_offset;    /* [B] position id of the root; NULL = 0 */
  void *event_between;          /* optional cudaEvent_t recorded on the stream between the V-wide kernel of step
                                   a1 and the tree kernel (ubt_draft_tree only; for timing the two apart -- an
                                   event between them also keeps the second from becoming resident early) */
  int32_t *status;              /* optional [B] device words, written for every sequence: 0, or UBT_STATUS_* bits
                                   (ubt_draft_tree: NaN / +inf among the unigram logits; ubt_build_tree: among the
                                   candidate log-probabilities it is given) */
  int32_t validate_finite;      /* host-buffer form only: return UBT_ERR_NONFINITE if any sequence was flagged */
} ubt_draft_opts;

typedef struct ubt_verify_opts {
  uint64_t seed;       /* Philox4x32-10 key (low word, high word); sampling mode only */
  float temperature;   /* > 0; sampling mode only; default 1 */
  int32_t *node_pick;  /* optional [B,N]: the target's pick at EVERY row, visited or not */
  void *event_before;  /* optional cudaEvent_t recorded on the stream just before the V-wide */
  void *event_after;   /* per-node kernel and just after it (for timing that kernel alone)    */
  int32_t early_start; /* 0 (default): plain stream order -- nothing is read or written before the work in
                          front of the call on `cuda_stream` has completed.  1: the caller vouches that
                          target_logits were complete, and the workspace and node_pick unused, BEFORE the
                          preceding ubt_draft_tree call on this stream was enqueued; the V-wide pass over
                          target_logits may then run while that draft call is still executing (it still
                          finishes after it, and the walk reads the finished tree).  Ignored -- the call falls
                          back to stream order -- when the stream's last draft call is not on record (the
                          library remembers the last one of 16 streams) or one of its buffers overlaps the
                          workspace or node_pick.  In the method's real order the target logits are computed
                          FROM the drafted tree (Appendix A), so leave this 0 there. */
  int32_t *status;     /* optional [B] device words, written for every sequence: 0, or UBT_STATUS_* bits (a NaN
                          or +inf in one of the sequence's N target rows, used slot or not) */
  int32_t validate_finite; /* host-buffer form only: return UBT_ERR_NONFINITE if any sequence was flagged */
  int32_t path_only;   /* 1: evaluate only the target rows the walk visits (at most L + 1 of the N rows of a
                          sequence) instead of all of them: the same verdict from a fraction of the bytes, as a
                          chain of at most L + 1 dependent steps inside one launch (a thread-block cluster per
                          sequence; no workspace is used, any B).  node_pick then receives the picks of the
                          visited slots and -1 elsewhere, status flags a NaN or +inf in a VISITED row only;
                          early_start is ignored.  Worth it when B * N is large (most rows are never visited);
                          for a single small tree the all-rows pass is as fast. */
} ubt_verify_opts;

typedef struct ubt_verify_result {
  int32_t *accepted_len;   /* [B]     accepted draft tokens; the paper's tau = accepted_len + 1 */
  int32_t *bonus_token;    /* [B]     first unmatched target pick */
  int32_t *accepted_nodes; /* [B,L+1] slots on the accepted path, root first; padded with -1 */
  int32_t *out_tokens;     /* [B,L+1] accepted tokens followed by the bonus token; padded with -1 */
} ubt_verify_result;

int ubt_version(void);
const char *ubt_status_string(int status);
/* Diagnostics: how many bounded device-side waits (on a bulk copy's completion) gave up since the library
 * was loaded on the current device.  0 in a healthy process; -1 if the counter cannot be read.  Results of a
 * call during which a wait gave up are undefined (but the call returned and nothing hung); the sequences
 * concerned carry UBT_STATUS_WAIT_GAVE_UP in the call's status words. */
long long ubt_debug_ring_timeouts(void);

/* Bytes of device workspace the calls below need for the given shape (0 on invalid shapes). */
size_t ubt_draft_workspace_bytes(int B, int L, int V, int k, int node_budget);
size_t ubt_verify_workspace_bytes(int B, int node_budget, int V, int mode);

/*
 * Step a1 alone (eq. 3 and "Candidate Sets", Section 3.1.1).  For each of `rows` logit rows of
 * length V: the k largest logits ordered (value descending, token id ascending; -0 equals +0),
 * and cand_logprob[r] = logit[cand_ids[r]] - log(sum_v exp logit[v]) in fp32.
 * Workspace: ubt_draft_workspace_bytes(rows, 1, V, k, 1).
 */
int ubt_topk_logprob(const void *logits, int dtype, int64_t rows, int V, int k, int32_t *cand_ids,
                     float *cand_logprob, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Step a1 with the vocabulary split over the ranks of a tensor-parallel group (the paper serves with the LM
 * head, and so every logits row, sharded over the vocabulary; Section 3.1.1 defines the candidates on the whole
 * row).  Rank r holds the columns [v0, v0 + Vs) of every row as a dense [rows, Vs] tensor and calls
 * ubt_topk_shard, which writes its per-row partial: (max, sum of exp relative to it), the k best values of the
 * slice (raw logits, best first) with their token ids in the WHOLE vocabulary (column + v0), and how many there
 * are.  The partial is one buffer of ubt_topk_shard_bytes(rows, k) bytes (the same for every rank; four arrays,
 * each 256-byte aligned: float[rows,2], float[rows,k], int32[rows,k], int32[rows]).  The caller gathers the
 * partials of all ranks back to back in rank order -- one all-gather of rows * (8k + 12) bytes, padding aside --
 * and every rank calls ubt_topk_merge_shards on the gathered buffer, which gives cand_ids / cand_logprob exactly
 * as ubt_topk_logprob would on the whole rows (same ordering, ties to the lower token id; the log-sum-exp is
 * summed in a different order, so log-probabilities agree to fp32 rounding).  Slices may differ in width; every
 * slice needs Vs >= k.  A slice whose streaming kernel gave up a wait has count -1 for the rows concerned; the
 * merge then treats its list as empty (ubt_debug_ring_timeouts tells).  No collective is issued by the library.
 * Workspace of ubt_topk_shard: ubt_draft_workspace_bytes(rows, 1, Vs, k, 1).
 */
size_t ubt_topk_shard_bytes(int64_t rows, int k);
int ubt_topk_shard(const void *logits_shard, int dtype, int64_t rows, int Vs, int k, int v0, void *partial,
                   void *workspace, size_t workspace_bytes, void *cuda_stream);
int ubt_topk_merge_shards(const void *gathered, int shards, int64_t rows, int k, int32_t *cand_ids,
                          float *cand_logprob, void *cuda_stream);

/*
 * The proposer's LM head fused with step a1 (Section 3.1.1, eq. 3: the unigram logits of a position are the
 * frozen LM head applied to the position's hidden state; the paper times this projection inside its draft
 * post-processing stage, appendix "Drafting Latency Analysis").  For each of `rows` hidden states:
 *   u[v] = sum_j hidden[row, j] * weight[v, j]          (bf16 inputs, fp32 accumulation on the tensor cores)
 * then the k largest u ordered (value descending, token id ascending) and cand_logprob[r] = u[cand_ids[r]] -
 * log(sum_v exp u[v]) -- the [rows, V] logits are never written to memory.  hidden: [rows, d] bf16 row-major;
 * weight: [V, d] bf16 row-major (one row of d weights per token); both 16-byte aligned, d a multiple of 64,
 * k <= 16 (else UBT_ERR_UNSUPPORTED: keep the logits and call ubt_topk_logprob).  The logits carry the
 * rounding of an fp32 accumulation in the tensor cores' order, so candidates whose logits differ by less than
 * about 1e-5 * sqrt(d) relative may come out in either order.  Workspace: ubt_lm_head_workspace_bytes().
 * A device-side wait that gives up (counted by ubt_debug_ring_timeouts) leaves the outputs undefined.
 */
size_t ubt_lm_head_workspace_bytes(int64_t rows, int d, int V, int k);
/*
 * The same with the head split over the ranks of a tensor-parallel group along the vocabulary, as the paper serves
 * it: weight_shard is this rank's [Vs, d] rows of the head (tokens v0 ... v0 + Vs - 1).  Writes this rank's per-row
 * partial in the format of ubt_topk_shard (ubt_topk_shard_bytes(rows, k) bytes: (max, sum exp), the k best raw
 * logits of the slice with token ids of the whole vocabulary, the count; k <= Vs); after one all-gather
 * ubt_topk_merge_shards gives every rank the candidates of the whole vocabulary.  Workspace:
 * ubt_lm_head_workspace_bytes(rows, d, Vs, k).
 */
int ubt_lm_head_topk_shard(const void *hidden, const void *weight_shard, int64_t rows, int d, int Vs, int k, int v0,
                           void *partial, void *workspace, size_t workspace_bytes, void *cuda_stream);
int ubt_lm_head_topk(const void *hidden, const void *weight, int64_t rows, int d, int V, int k, int32_t *cand_ids,
                     float *cand_logprob, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Steps a2, a3, a3b from candidates that are already in out->cand_ids / out->cand_logprob
 * (eq. 5, eq. 9-12, Algorithm 1).  bigram_scores[b,j,ra,rb] is the selector score delta of the
 * transition from the rank-ra candidate of position j to the rank-rb candidate of position j+1.
 * s = alpha*logprob + lambda*delta is normalised over the k successor candidates of each
 * predecessor; a node's score is the sum of those log-probabilities along its prefix plus
 * zeta*depth.  The search keeps, per depth, the W best extensions of the retained nodes and
 * finally the N-1 best retained nodes overall; ties prefer the shallower node, then the lower
 * token id, then the lower candidate rank, then the lexicographically smaller rank path.
 * Scores are computed in fp32.
 */
int ubt_build_tree(const float *bigram_scores, int B, int L, int k, int node_budget,
                   const ubt_draft_opts *opts, ubt_tree *out, void *cuda_stream);

/*
 * The step between a1 and a2 in the paper's data flow (Section 3.1.2, "Parallel Computation": the
 * edge matrix Delta_i = Phi_{i-1} diag(P(h_i)) Psi_i^T): the selector score of every
 * (predecessor candidate, successor candidate) pair from the precomputed codebook tables,
 *   delta_i(a, b) = sum_r gate[b, i, r] * phi[a, r] * psi[b, r].
 * phi, psi: [V, R] row-major device tables of `table_dtype` (ubt_dtype), 16-byte aligned, R a
 * multiple of 8 (bf16) / 4 (fp32), R <= 8192; gate: [B, L, R] fp32, the projected proposer
 * state P(h_i) of each position; cand_ids: [B, L, k] as written by ubt_topk_logprob (every id in
 * [0, V); ids outside give unspecified but memory-safe scores).  Writes
 *   bigram_scores[b, j, ra, rb] (j < L-1): rank-ra candidate of position j -> rank-rb candidate of
 *     position j+1, gate of position j+1                              ([B, L-1, k, k] fp32), and,
 *   if anchor_tokens and anchor_bigram are both non-NULL, anchor_bigram[b, rb]: anchor token ->
 *     rank-rb candidate of position 0, gate of position 0             ([B, k] fp32),
 * i.e. exactly the selector inputs of ubt_build_tree.  Products and sums are fp32 (fma) in the
 * order of r; results agree with a double-precision sum to about 1e-6 * sum_r |term|.  No workspace.  Errors as for the other calls.
 */
int ubt_selector_scores(const void *phi, const void *psi, int table_dtype, int V, int R,
                        const float *gate, const int32_t *cand_ids,
                        const int32_t *anchor_tokens /* [B] or NULL */, int B, int L, int k,
                        float *bigram_scores, float *anchor_bigram /* [B,k] or NULL */,
                        void *cuda_stream);

/*
 * Step a3b alone: position ids and the ancestor bitmask from parents / depths / n_nodes of `tree`
 * (for callers that edit a tree).  Overwrites tree->position_ids and tree->mask.
 */
int ubt_build_mask(ubt_tree *tree, const int32_t *pos_offset /* [B] or NULL */, void *cuda_stream);

/*
 * Steps a1 -> a3b in one call: unigram_logits[B,L,V] (fp32 or bf16) and bigram_scores[B,L-1,k,k]
 * (fp32) -> *out.  Equivalent to ubt_topk_logprob followed by ubt_build_tree.
 */
int ubt_draft_tree(const void *unigram_logits, int dtype, const float *bigram_scores, int B, int L,
                   int V, int k, int node_budget, const ubt_draft_opts *opts, ubt_tree *out,
                   void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Step a4 (Appendix A, "Verification via Tree-attention").  target_logits[B,N,V] holds one row per
 * tree slot.  The target's pick at a row is, in greedy mode, the smallest token id attaining the
 * row maximum; in sampling mode, a draw from softmax(row / temperature) defined by integer
 * weights w_v = trunc(2^(40 + fma(z_v, a, c))) (a = log2(e)/T, c = -max*a, a fixed fp32 degree-5
 * routine for 2^x), theta = floor(R * sum(w) / 2^64) with R the first two words of
 * Philox4x32-10(counter = (slot, b, 0, 0), key = seed), pick = first token whose inclusive prefix
 * sum exceeds theta.  The walk starts at the root and follows the child whose token equals the pick
 * of the current slot until none matches; that pick is the bonus token.
 */
int ubt_verify_tree(const ubt_tree *tree, const void *target_logits, int dtype, int V, int mode,
                    const ubt_verify_opts *opts, ubt_verify_result *out, void *workspace,
                    size_t workspace_bytes, void *cuda_stream);

/*
 * Greedy step a4 with the vocabulary of the target logits split over the ranks of a tensor-parallel group
 * (appendix "Verification via Tree-attention": the pick of a slot is the arg max over the whole vocabulary).
 * Rank r holds the columns [v0, v0 + Vs) of every target row as a dense [B, node_budget, Vs] tensor and calls
 * ubt_verify_keys_shard, which writes one 8-byte ordering key per row into row_keys[B * node_budget]: the best
 * (value, token) of the slice with the token counted in the WHOLE vocabulary; a larger key is a better pick
 * (higher value, then lower token id), so the pick of a row is the maximum of the ranks' keys.  The caller
 * gathers the ranks' key arrays back to back in rank order (one all-gather of B * node_budget * 8 bytes) and
 * every rank calls ubt_verify_tree_keys, which takes the maximum per slot and walks the tree exactly as
 * ubt_verify_tree does in greedy mode: identical accepted_len, accepted_nodes, out_tokens, bonus_token,
 * node_pick and status words (a NaN, +inf or an abandoned wait in any slice is reported).  Of `opts` only
 * node_pick and status are read.  Workspace of ubt_verify_keys_shard: ubt_verify_workspace_bytes(B,
 * node_budget, Vs, UBT_VERIFY_GREEDY).  No collective is issued by the library.  Sampling is not split this way.
 */
int ubt_verify_keys_shard(const void *target_shard, int dtype, int B, int node_budget, int Vs, int v0,
                          unsigned long long *row_keys, void *workspace, size_t workspace_bytes,
                          void *cuda_stream);
int ubt_verify_tree_keys(const ubt_tree *tree, const unsigned long long *gathered_keys, int shards,
                         ubt_verify_result *out, const ubt_verify_opts *opts, void *cuda_stream);

/*
 * The walk of step a4 alone (Appendix A, "Verification via Tree-attention"), for callers that already hold the
 * target's pick of every slot.  node_pick[B, node_budget] (DEVICE, int32, read only) is the token the target
 * chose at each slot: from ubt_lm_head_topk with k = 1 on the target's hidden states of the tree slots (greedy
 * verification with the target logits never written to memory: cand_ids[B * node_budget, 1] IS this array), from
 * a sampler of the caller's, or gathered from the ranks of a vocabulary-parallel group: with shards > 1 node_pick
 * is [shards, B, node_budget] and the pick of a slot is the largest of the shards' entries (the rank that owns the
 * pick holds a token, the others -1; if all are negative the smallest is taken); shards = 1 otherwise.  From the
 * root the walk follows the child whose token equals the pick of the current slot until none matches; that pick is
 * the bonus token.  *out is written as ubt_verify_tree writes it.  Every entry must be a token id >= 0 or negative
 * for "no valid pick": a sequence with a negative pick at any of its node_budget slots gets UBT_STATUS_NONFINITE
 * (UBT_STATUS_WAIT_GAVE_UP for -2) in status[b] (DEVICE, B words, may be NULL), and the pick counts as token 0.
 * No workspace.  Stream-ordered like every other call.
 */
int ubt_verify_tree_picks(const ubt_tree *tree, const int32_t *node_pick, int shards, ubt_verify_result *out,
                          int32_t *status, void *cuda_stream);

/*
 * Sampling step a4 with the vocabulary of the target logits split over the ranks of a tensor-parallel group.  The
 * integer weights of ubt_verify_tree's sampling mode make the split exact -- the picks are bit-identical to those
 * of one GPU holding whole rows.  Rank r holds the columns [v0, v0 + Vs) of every target row as a dense
 * [B, node_budget, Vs] tensor; ranks are numbered in the order of their columns.  Per call of the verifier:
 *   1. ubt_verify_keys_shard (above) -> row_keys; all-gather -> gathered_keys[shards, B * node_budget]: the row
 *      maximum over the whole vocabulary is the value of the largest key;
 *   2. ubt_sample_totals_shard: the weights w_v = trunc(2^(40 + fma(z_v, a, c))) of this rank's columns with
 *      a = log2(e)/temperature, c = -max * a, summed per row into totals[B * node_budget] (DEVICE, uint64); the
 *      per-1024-token sums stay in `workspace` for step 3; all-gather -> gathered_totals[shards, B * node_budget];
 *   3. ubt_sample_picks_shard: theta = floor(R * sum of the ranks' totals / 2^64) as in ubt_verify_tree; the one
 *      rank whose share of the running sum over ranks holds theta writes the token (counted in the WHOLE
 *      vocabulary) to picks[B * node_budget] (DEVICE, int32), every other rank -1; a row whose maximum is NaN or
 *      +inf on any rank gets -1 from every rank (-2 after an abandoned device-side wait);
 *      all-gather -> gathered_picks[shards, B * node_budget];
 *   4. ubt_verify_tree_picks with that array and `shards`.
 * `workspace` (steps 2 and 3, the same buffer, untouched in between): ubt_verify_workspace_bytes(B, node_budget, Vs,
 * UBT_VERIFY_SAMPLE).  `rank` is this rank's position in the gathered arrays.  No collective is issued by the
 * library: three all-gathers of 8, 8 and 4 bytes per tree slot.
 */
int ubt_sample_totals_shard(const void *target_shard, int dtype, int B, int node_budget, int Vs,
                            const unsigned long long *gathered_keys, int shards, float temperature,
                            unsigned long long *totals, void *workspace, size_t workspace_bytes,
                            void *cuda_stream);
int ubt_sample_picks_shard(const void *target_shard, int dtype, int B, int node_budget, int Vs, int v0, int rank,
                           const unsigned long long *gathered_totals, int shards, uint64_t seed, int32_t *picks,
                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Host-buffer forms.  Every pointer inside `tree`, `opts` (alpha ... pos_offset, node_pick) and
 * `out`, and the logits / bigram arguments, are HOST pointers (pinned memory makes the copies
 * asynchronous).  `device_buffer` is caller-owned DEVICE memory of at least
 * ubt_*_host_buffer_bytes(); the call copies inputs into it, runs the device path on
 * `cuda_stream`, copies the results back and waits for the stream before returning.
 */
size_t ubt_draft_host_buffer_bytes(int B, int L, int V, int k, int node_budget, int dtype);
size_t ubt_verify_host_buffer_bytes(int B, int L, int node_budget, int V, int dtype, int mode);
int ubt_draft_tree_host(const void *unigram_logits, int dtype, const float *bigram_scores, int B,
                        int L, int V, int k, int node_budget, const ubt_draft_opts *opts,
                        ubt_tree *out, void *device_buffer, size_t device_buffer_bytes,
                        void *cuda_stream);
int ubt_verify_tree_host(const ubt_tree *tree, const void *target_logits, int dtype, int V, int mode,
                         const ubt_verify_opts *opts, ubt_verify_result *out, void *device_buffer,
                         size_t device_buffer_bytes, void *cuda_stream);

/*
 * Greedy verification for callers that cannot allocate device memory (the paper has no counterpart: this
 * is a packaging variant of ubt_verify_tree in UBT_VERIFY_GREEDY mode).  Such callers are, for example,
 * code running after a memory pool has handed out all of the device, a plugin that only ever receives its
 * input and output buffers, or a latency-critical loop that must not hit cudaMalloc's implicit
 * synchronisation.  The call takes no workspace: its scratch (one 8-byte key per row and span) lives in a
 * 512 KiB array compiled into the library, which every GPU that loads the library holds until the process
 * ends.  It allocates nothing, frees nothing and calls no allocating routine.
 *
 * Same arguments, outputs and results as ubt_verify_tree(tree, target_logits, dtype, V, GREEDY, ...);
 * node_pick ([B,N] device, may be NULL) receives the pick of every row.
 * Limit: B*N*spans_per_row <= ubt_verify_static_capacity() keys (65,536), where spans_per_row =
 * ceil(V/span)+1 and span = max(32,768, ceil(B*N*V / SM count)) elements rounded up to a multiple of 256:
 * 2 for large batches (32,768 keys for B*N = 16,384 rows), 4 for a single 64-slot tree over V = 151,936
 * on 148 SMs.  A larger request returns UBT_ERR_STATIC_SCRATCH before anything is launched.
 * The first call on a device looks up the array's device address (once per device, with that device
 * current); make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents (every key that is
 * read is written first, so nothing needs clearing).  Calls enqueued one after the other on the SAME stream
 * are safe: the call keeps plain stream order, so its first kernel starts only after the walk of the call in
 * front has finished with the array.  Two calls whose kernels can overlap on the GPU -- different streams, or
 * different host threads enqueueing without an order between them -- race on it and must be serialised by
 * the caller.
 */
int ubt_verify_tree_static(const ubt_tree *tree, const void *target_logits, int dtype, int V,
                           int32_t *node_pick, ubt_verify_result *out, void *cuda_stream);
long long ubt_verify_static_capacity(void);

#ifdef __cplusplus
}
#endif
#endif /* UBT_H_ */
