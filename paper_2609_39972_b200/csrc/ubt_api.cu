// C ABI of libubt: argument validation, workspace carving, launches.  See include/ubt.h.
#include <cstring>
#include <mutex>
#include <new>

#include "ubt_internal.h"

namespace ubt {

const DeviceInfo& device_info() {
  static DeviceInfo info[64];
  static bool known[64];
  static std::mutex mu;
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 0 || dev >= 64) dev = 0;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[dev]) {
    int sms = 0, smem = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    if (cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess || smem <= 0)
      smem = 227 * 1024;
    cudaGetLastError();
    info[dev].device = dev;
    info[dev].sm_count = sms;
    info[dev].max_smem_optin = smem;
    known[dev] = true;
  }
  return info[dev];
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static size_t esize(int dtype) { return dtype == UBT_BF16 ? 2 : 4; }

static int check_shape(int B, int L, int V, int k, int N) {
  if (B < 0 || L < 1 || V < 1 || k < 1 || N < 1 || k > V) return UBT_ERR_INVALID_ARG;
  if (k > kMaxK || N > kMaxN || L > kMaxL) return UBT_ERR_UNSUPPORTED;
  return UBT_OK;
}

static int check_tree(const ubt_tree* t, bool need_cands) {
  if (!t) return UBT_ERR_INVALID_ARG;
  if (t->mask_words != (t->N + 31) / 32) return UBT_ERR_INVALID_ARG;
  const void* ptrs[] = {t->token_ids, t->parents, t->depths, t->position_ids, t->cand_rank,
                        t->scores,    t->mask,    t->n_nodes};
  for (const void* p : ptrs)
    if (!p || !aligned16(p)) return UBT_ERR_INVALID_ARG;
  if (need_cands && (!t->cand_ids || !t->cand_logprob || !aligned16(t->cand_ids) || !aligned16(t->cand_logprob)))
    return UBT_ERR_INVALID_ARG;
  return UBT_OK;
}

// ---- which memory a draft call on a stream may still be using when the next call starts
//
// A verify call keeps plain stream order unless the caller sets ubt_verify_opts.early_start; then its V-wide
// pass streams while the draft call in front of it on the stream is still running.  Beyond what the caller
// vouches for (the target logits were complete before that draft call was enqueued), this is only sound if
// nothing the early kernel WRITES overlaps anything the draft call reads or writes; plain stream order would
// allow such reuse (say, the draft logits' buffer as the verify workspace).  Every draft call therefore records
// its buffers per stream, and an early start is granted only against a recorded draft call that the written
// buffers stay clear of.
struct ByteRange {
  const char* lo;
  const char* hi;
};
struct DraftRecord {
  cudaStream_t stream;
  bool valid;
  int n;
  ByteRange r[24];
};
static std::mutex g_draft_mu;
static DraftRecord g_drafts[16];
static unsigned g_draft_next;

static void add_range(DraftRecord& d, const void* p, size_t bytes) {
  if (p && bytes && d.n < 24) d.r[d.n++] = ByteRange{static_cast<const char*>(p), static_cast<const char*>(p) + bytes};
}

static void remember_draft(cudaStream_t st, const void* logits, size_t logits_bytes, const float* bigram, int B, int L,
                           int k, int N, const ubt_draft_opts* o, const ubt_tree& t, const void* ws, size_t ws_bytes) {
  DraftRecord d{};
  d.stream = st;
  d.valid = true;
  const size_t bn = (size_t)B * N, blk = (size_t)B * L * k;
  add_range(d, logits, logits_bytes);
  add_range(d, bigram, (size_t)B * (L > 1 ? L - 1 : 0) * k * k * 4);
  add_range(d, ws, ws_bytes);
  if (o) {
    add_range(d, o->alpha, (size_t)L * 4);
    add_range(d, o->lambda, (size_t)L * 4);
    add_range(d, o->anchor_bigram, (size_t)B * k * 4);
    add_range(d, o->anchor_tokens, (size_t)B * 4);
    add_range(d, o->pos_offset, (size_t)B * 4);
    add_range(d, o->status, (size_t)B * 4);
  }
  const void* per_node[] = {t.token_ids, t.parents, t.depths, t.position_ids, t.cand_rank, t.scores};
  for (const void* p : per_node) add_range(d, p, bn * 4);
  add_range(d, t.mask, bn * t.mask_words * 4);
  add_range(d, t.n_nodes, (size_t)B * 4);
  add_range(d, t.cand_ids, blk * 4);
  add_range(d, t.cand_logprob, blk * 4);
  std::lock_guard<std::mutex> lock(g_draft_mu);
  for (DraftRecord& e : g_drafts)
    if (e.valid && e.stream == st) { e = d; return; }
  g_drafts[g_draft_next++ % 16] = d;
}

// May a kernel that writes [p, p + bytes) start while the last draft call on `st` is still running?  Only if
// that call is on record (the table holds the last draft of 16 streams; a stream that was pushed out of it, or
// never drafted, gets the answer "no") and none of its buffers overlaps the range.
static bool clear_of_last_draft(cudaStream_t st, const void* p, size_t bytes) {
  const char* lo = static_cast<const char*>(p);
  const char* hi = lo + (p ? bytes : 0);
  std::lock_guard<std::mutex> lock(g_draft_mu);
  for (const DraftRecord& e : g_drafts) {
    if (!e.valid || e.stream != st) continue;
    for (int i = 0; i < e.n; ++i)
      if (lo < e.r[i].hi && e.r[i].lo < hi) return false;
    return true;
  }
  return false;
}

}  // namespace ubt

using namespace ubt;

extern "C" {

int ubt_version(void) { return 110; }

const char* ubt_status_string(int status) {
  switch (status) {
    case UBT_OK: return "ok";
    case UBT_ERR_INVALID_ARG: return "invalid argument";
    case UBT_ERR_UNSUPPORTED: return "shape beyond the compiled limits";
    case UBT_ERR_WORKSPACE: return "workspace missing or too small";
    case UBT_ERR_CUDA: return "CUDA call or launch failed";
    case UBT_ERR_STATIC_SCRATCH: return "request exceeds the built-in scratch of ubt_verify_tree_static";
    case UBT_ERR_NONFINITE: return "NaN or +inf among the logits";
    default: return "unknown status";
  }
}

size_t ubt_draft_workspace_bytes(int B, int L, int V, int k, int N) {
  if (B < 0 || L < 1 || V < 1 || k < 1 || N < 1 || k > V || k > kMaxK) return 0;
  return topk_workspace_bytes((int64_t)B * L, V, k) + 256;
}

size_t ubt_verify_workspace_bytes(int B, int N, int V, int mode) {
  if (B < 0 || N < 1 || V < 1 || (mode != UBT_VERIFY_GREEDY && mode != UBT_VERIFY_SAMPLE)) return 0;
  const size_t all_rows = verify_workspace_bytes((int64_t)B * N, V, mode), path = verify_path_workspace_bytes(B, N, mode);
  return (all_rows > path ? all_rows : path) + 256;  // either form of the call fits
}

int ubt_topk_logprob(const void* logits, int dtype, int64_t rows, int V, int k, int32_t* cand_ids,
                     float* cand_logprob, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!logits || !cand_ids || !cand_logprob || rows < 0 || V < 1 || k < 1 || k > V) return UBT_ERR_INVALID_ARG;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!aligned16(logits) || !aligned16(cand_ids) || !aligned16(cand_logprob)) return UBT_ERR_INVALID_ARG;
  if (k > kMaxK) return UBT_ERR_UNSUPPORTED;
  if (rows == 0) return UBT_OK;
  if (!workspace || !aligned16(workspace) || workspace_bytes < topk_workspace_bytes(rows, V, k))
    return UBT_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  TopkWorkspace w = carve_topk_workspace(workspace, rows, V, k);
  if (launch_lse_topk(logits, dtype, rows, V, k, w, st) != cudaSuccess) return UBT_ERR_CUDA;
  if (launch_merge_topk(rows, V, k, w, cand_ids, cand_logprob, st) != cudaSuccess) return UBT_ERR_CUDA;
  return UBT_OK;
}

size_t ubt_topk_shard_bytes(int64_t rows, int k) {
  if (rows < 0 || k < 1 || k > kMaxK) return 0;
  return shard_partial_bytes(rows, k);
}

int ubt_topk_shard(const void* logits_shard, int dtype, int64_t rows, int Vs, int k, int v0, void* partial,
                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!logits_shard || !partial || rows < 0 || Vs < 1 || k < 1 || k > Vs || v0 < 0) return UBT_ERR_INVALID_ARG;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!aligned16(logits_shard) || !aligned16(partial)) return UBT_ERR_INVALID_ARG;
  if (k > kMaxK || (int64_t)v0 + Vs > 0x7fffffffll) return UBT_ERR_UNSUPPORTED;
  if (rows == 0) return UBT_OK;
  if (!workspace || !aligned16(workspace) || workspace_bytes < topk_workspace_bytes(rows, Vs, k))
    return UBT_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  TopkWorkspace w = carve_topk_workspace(workspace, rows, Vs, k);
  if (launch_lse_topk(logits_shard, dtype, rows, Vs, k, w, st) != cudaSuccess) return UBT_ERR_CUDA;
  const cudaError_t e = launch_merge_topk_shard(rows, Vs, k, w, partial, v0, st);
  if (e != cudaSuccess) { cudaGetLastError(); return e == cudaErrorNotSupported ? UBT_ERR_UNSUPPORTED : UBT_ERR_CUDA; }
  return UBT_OK;
}

int ubt_topk_merge_shards(const void* gathered, int shards, int64_t rows, int k, int32_t* cand_ids,
                          float* cand_logprob, void* cuda_stream) {
  if (!gathered || !cand_ids || !cand_logprob || shards < 1 || rows < 0 || k < 1) return UBT_ERR_INVALID_ARG;
  if (!aligned16(gathered) || !aligned16(cand_ids) || !aligned16(cand_logprob)) return UBT_ERR_INVALID_ARG;
  if (k > kMaxK) return UBT_ERR_UNSUPPORTED;
  if (rows == 0) return UBT_OK;
  const cudaError_t e = launch_merge_shards(gathered, shards, rows, k, cand_ids, cand_logprob,
                                            static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) { cudaGetLastError(); return e == cudaErrorNotSupported ? UBT_ERR_UNSUPPORTED : UBT_ERR_CUDA; }
  return UBT_OK;
}

size_t ubt_lm_head_workspace_bytes(int64_t rows, int d, int V, int k) {
  if (rows < 0 || d < 1 || V < 1 || k < 1 || k > V || k > lm_head_max_k() || d % 64 != 0 || rows > lm_head_max_rows())
    return 0;
  return lm_head_workspace_bytes(rows, k);
}

int ubt_lm_head_topk(const void* hidden, const void* weight, int64_t rows, int d, int V, int k, int32_t* cand_ids,
                     float* cand_logprob, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!hidden || !weight || !cand_ids || !cand_logprob || rows < 0 || d < 1 || V < 1 || k < 1 || k > V)
    return UBT_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(weight) || !aligned16(cand_ids) || !aligned16(cand_logprob))
    return UBT_ERR_INVALID_ARG;
  if (d % 64 != 0 || k > lm_head_max_k() || rows > lm_head_max_rows() || device_info().sm_count > 256)
    return UBT_ERR_UNSUPPORTED;
  if (rows == 0) return UBT_OK;
  if (!workspace || !aligned16(workspace) || workspace_bytes < lm_head_workspace_bytes(rows, k)) return UBT_ERR_WORKSPACE;
  cudaError_t e = launch_lm_head_topk(hidden, weight, rows, d, V, k, cand_ids, cand_logprob, workspace,
                                      static_cast<cudaStream_t>(cuda_stream));
  if (e != cudaSuccess) { cudaGetLastError(); return e == cudaErrorNotSupported ? UBT_ERR_UNSUPPORTED : UBT_ERR_CUDA; }
  return UBT_OK;
}

int ubt_lm_head_topk_shard(const void* hidden, const void* weight_shard, int64_t rows, int d, int Vs, int k, int v0,
                           void* partial, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!hidden || !weight_shard || !partial || rows < 0 || d < 1 || Vs < 1 || k < 1 || k > Vs || v0 < 0)
    return UBT_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(weight_shard) || !aligned16(partial)) return UBT_ERR_INVALID_ARG;
  if (d % 64 != 0 || k > lm_head_max_k() || rows > lm_head_max_rows() || device_info().sm_count > 256 ||
      (int64_t)v0 + Vs > 0x7fffffffll)
    return UBT_ERR_UNSUPPORTED;
  if (rows == 0) return UBT_OK;
  if (!workspace || !aligned16(workspace) || workspace_bytes < lm_head_workspace_bytes(rows, k)) return UBT_ERR_WORKSPACE;
  cudaError_t e = launch_lm_head_topk(hidden, weight_shard, rows, d, Vs, k, nullptr, nullptr, workspace,
                                      static_cast<cudaStream_t>(cuda_stream), partial, v0);
  if (e != cudaSuccess) { cudaGetLastError(); return e == cudaErrorNotSupported ? UBT_ERR_UNSUPPORTED : UBT_ERR_CUDA; }
  return UBT_OK;
}

static int check_draft_opts(const ubt_draft_opts* o) {
  if (!o) return UBT_OK;
  if (o->search_width < 0 || !(o->depth_bonus <= 0.0f)) return UBT_ERR_INVALID_ARG;
  return UBT_OK;
}

int ubt_build_tree(const float* bigram_scores, int B, int L, int k, int N, const ubt_draft_opts* opts,
                   ubt_tree* out, void* cuda_stream) {
  int rc = check_shape(B, L, k, k, N);  // V is not an input here; k stands in for the k <= V check
  if (rc) return rc;
  if ((rc = check_tree(out, true))) return rc;
  if ((rc = check_draft_opts(opts))) return rc;
  if (L > 1 && (!bigram_scores || !aligned16(bigram_scores))) return UBT_ERR_INVALID_ARG;
  if (out->B != B || out->N != N || out->L != L || out->k != k) return UBT_ERR_INVALID_ARG;
  if (tree_smem_bytes(L, k, N) > (size_t)device_info().max_smem_optin) return UBT_ERR_UNSUPPORTED;
  const ubt_draft_opts d{};
  const ubt_draft_opts* o = opts ? opts : &d;
  remember_draft(static_cast<cudaStream_t>(cuda_stream), nullptr, 0, bigram_scores, B, L, k, N, o, *out, nullptr, 0);
  cudaError_t e = launch_build_tree(bigram_scores, B, L, k, N, o->search_width, o->depth_bonus, o->alpha, o->lambda,
                                    o->anchor_bigram, o->anchor_tokens, o->pos_offset, *out, no_merge_parts(), 0,
                                    o->status, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? UBT_OK : UBT_ERR_CUDA;
}

int ubt_selector_scores(const void* phi, const void* psi, int table_dtype, int V, int R, const float* gate,
                        const int32_t* cand_ids, const int32_t* anchor_tokens, int B, int L, int k,
                        float* bigram_scores, float* anchor_bigram, void* cuda_stream) {
  if (B < 0 || L < 1 || V < 1 || k < 1 || R < 1) return UBT_ERR_INVALID_ARG;
  if (table_dtype != UBT_F32 && table_dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!phi || !psi || !gate || !cand_ids || !aligned16(phi) || !aligned16(psi)) return UBT_ERR_INVALID_ARG;
  if (L > 1 && !bigram_scores) return UBT_ERR_INVALID_ARG;
  if ((anchor_bigram != nullptr) != (anchor_tokens != nullptr)) return UBT_ERR_INVALID_ARG;
  if (R % (table_dtype == UBT_BF16 ? 8 : 4) != 0) return UBT_ERR_INVALID_ARG;
  if (k > kMaxK || L > kMaxL || R > kMaxSelectorRank) return UBT_ERR_UNSUPPORTED;
  cudaError_t e = launch_selector_scores(phi, psi, table_dtype, V, R, gate, cand_ids, anchor_tokens, B, L, k,
                                         bigram_scores, anchor_bigram, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? UBT_OK : UBT_ERR_CUDA;
}

int ubt_build_mask(ubt_tree* tree, const int32_t* pos_offset, void* cuda_stream) {
  int rc = check_tree(tree, false);
  if (rc) return rc;
  if (tree->B < 0 || tree->N < 1) return UBT_ERR_INVALID_ARG;
  if (tree->N > kMaxN) return UBT_ERR_UNSUPPORTED;
  cudaError_t e = launch_build_mask(*tree, pos_offset, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? UBT_OK : UBT_ERR_CUDA;
}

int ubt_draft_tree(const void* unigram_logits, int dtype, const float* bigram_scores, int B, int L, int V, int k,
                   int N, const ubt_draft_opts* opts, ubt_tree* out, void* workspace, size_t workspace_bytes,
                   void* cuda_stream) {
  int rc = check_shape(B, L, V, k, N);
  if (rc) return rc;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!unigram_logits || !aligned16(unigram_logits)) return UBT_ERR_INVALID_ARG;
  if ((rc = check_tree(out, true))) return rc;
  if ((rc = check_draft_opts(opts))) return rc;
  if (L > 1 && (!bigram_scores || !aligned16(bigram_scores))) return UBT_ERR_INVALID_ARG;
  if (out->B != B || out->N != N || out->L != L || out->k != k) return UBT_ERR_INVALID_ARG;
  if (tree_smem_bytes(L, k, N) > (size_t)device_info().max_smem_optin) return UBT_ERR_UNSUPPORTED;
  if (B == 0) return UBT_OK;
  const int64_t rows = (int64_t)B * L;
  if (!workspace || !aligned16(workspace) || workspace_bytes < topk_workspace_bytes(rows, V, k))
    return UBT_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  TopkWorkspace w = carve_topk_workspace(workspace, rows, V, k);
  if (launch_lse_topk(unigram_logits, dtype, rows, V, k, w, st) != cudaSuccess) return UBT_ERR_CUDA;
  // the tree kernel merges the row partials in its prologue: one launch less than topk + merge + tree
  const ubt_draft_opts d{};
  const ubt_draft_opts* o = opts ? opts : &d;
  remember_draft(st, unigram_logits, (size_t)rows * V * esize(dtype), bigram_scores, B, L, k, N, o, *out, workspace,
                 topk_workspace_bytes(rows, V, k));
  if (o->event_between && cudaEventRecord(static_cast<cudaEvent_t>(o->event_between), st) != cudaSuccess)
    return UBT_ERR_CUDA;
  cudaError_t e = launch_build_tree(bigram_scores, B, L, k, N, o->search_width, o->depth_bonus, o->alpha, o->lambda,
                                    o->anchor_bigram, o->anchor_tokens, o->pos_offset, *out, merge_parts(w), V,
                                    o->status, st);
  return e == cudaSuccess ? UBT_OK : UBT_ERR_CUDA;
}

int ubt_verify_tree(const ubt_tree* tree, const void* target_logits, int dtype, int V, int mode,
                    const ubt_verify_opts* opts, ubt_verify_result* out, void* workspace, size_t workspace_bytes,
                    void* cuda_stream) {
  int rc = check_tree(tree, false);
  if (rc) return rc;
  if (!target_logits || !aligned16(target_logits) || !out || V < 1) return UBT_ERR_INVALID_ARG;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (mode != UBT_VERIFY_GREEDY && mode != UBT_VERIFY_SAMPLE) return UBT_ERR_INVALID_ARG;
  if (!out->accepted_len || !out->bonus_token || !out->accepted_nodes || !out->out_tokens) return UBT_ERR_INVALID_ARG;
  const int B = tree->B, N = tree->N, L = tree->L;
  if (B < 0 || N < 1 || L < 1) return UBT_ERR_INVALID_ARG;
  if (N > kMaxN || L > kMaxL) return UBT_ERR_UNSUPPORTED;
  const ubt_verify_opts d{0, 1.0f, nullptr, nullptr, nullptr, 0, nullptr, 0, 0};
  const ubt_verify_opts* o = opts ? opts : &d;
  if (mode == UBT_VERIFY_SAMPLE) {
    if (!(o->temperature > 0.0f)) return UBT_ERR_INVALID_ARG;
    if (V > 2048 * 1024) return UBT_ERR_UNSUPPORTED;
  }
  if (o->path_only && B > verify_path_max_batch()) return UBT_ERR_UNSUPPORTED;
  if (B == 0) return UBT_OK;
  const int64_t rows = (int64_t)B * N;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (o->path_only) {
    if (!workspace || !aligned16(workspace) || workspace_bytes < verify_path_workspace_bytes(B, N, mode))
      return UBT_ERR_WORKSPACE;
    if (o->event_before && cudaEventRecord(static_cast<cudaEvent_t>(o->event_before), st) != cudaSuccess)
      return UBT_ERR_CUDA;
    if (launch_verify_path(*tree, target_logits, dtype, V, mode, o->seed, o->temperature, workspace, o->node_pick, *out,
                           o->status, st) != cudaSuccess) {
      cudaGetLastError();
      return UBT_ERR_CUDA;
    }
    if (o->event_after && cudaEventRecord(static_cast<cudaEvent_t>(o->event_after), st) != cudaSuccess)
      return UBT_ERR_CUDA;
    return UBT_OK;
  }
  if (!workspace || !aligned16(workspace) || workspace_bytes < verify_workspace_bytes(rows, V, mode))
    return UBT_ERR_WORKSPACE;
  VerifyWorkspace w = carve_verify_workspace(workspace, rows, V, mode);
  const int32_t* sampled = nullptr;
  if (o->event_before && cudaEventRecord(static_cast<cudaEvent_t>(o->event_before), st) != cudaSuccess)
    return UBT_ERR_CUDA;
  // stream order by default; on request the V-wide kernels start while the draft call in front of them on this
  // stream is still running, unless what they write touches that call's buffers
  bool early = o->early_start != 0 && clear_of_last_draft(st, workspace, verify_workspace_bytes(rows, V, mode));
  if (mode == UBT_VERIFY_GREEDY) {
    if (launch_row_argmax(target_logits, dtype, rows, V, w, tree_smem_bytes(tree->L, tree->k, tree->N), early, st) !=
        cudaSuccess)
      return UBT_ERR_CUDA;
  } else {
    int32_t* pick = o->node_pick ? o->node_pick : w.pick;
    early = early && (!o->node_pick || clear_of_last_draft(st, o->node_pick, (size_t)rows * 4));
    if (launch_row_sample(target_logits, dtype, B, N, V, o->seed, o->temperature, pick, w, early, st) != cudaSuccess)
      return UBT_ERR_CUDA;
    sampled = pick;
  }
  if (o->event_after && cudaEventRecord(static_cast<cudaEvent_t>(o->event_after), st) != cudaSuccess)
    return UBT_ERR_CUDA;
  if (launch_walk(*tree, mode, w, V, sampled, o->node_pick, *out, o->status, st) != cudaSuccess) return UBT_ERR_CUDA;
  return UBT_OK;
}

int ubt_verify_tree_picks(const ubt_tree* tree, const int32_t* node_pick, int shards, ubt_verify_result* out,
                          int32_t* status, void* cuda_stream) {
  if (!tree || !out || !node_pick || shards < 1) return UBT_ERR_INVALID_ARG;
  if (!tree->token_ids || !tree->parents || !tree->n_nodes) return UBT_ERR_INVALID_ARG;
  if (!out->accepted_len || !out->bonus_token || !out->accepted_nodes || !out->out_tokens) return UBT_ERR_INVALID_ARG;
  const int B = tree->B, N = tree->N, L = tree->L;
  if (B < 0 || N < 1 || L < 1) return UBT_ERR_INVALID_ARG;
  if (N > kMaxN || L > kMaxL) return UBT_ERR_UNSUPPORTED;
  if (B == 0) return UBT_OK;
  // the walk kernel in the mode that takes the picks as given (the sampling mode's second half)
  if (launch_walk(*tree, UBT_VERIFY_SAMPLE, VerifyWorkspace{}, 0, node_pick, nullptr, *out, status,
                  static_cast<cudaStream_t>(cuda_stream), shards) != cudaSuccess)
    return UBT_ERR_CUDA;
  return UBT_OK;
}

static int check_sample_shard(const void* target_shard, int dtype, int B, int N, int Vs, const void* gathered, int shards,
                              void* workspace, size_t workspace_bytes) {
  if (!target_shard || !gathered || B < 0 || N < 1 || Vs < 1 || shards < 1) return UBT_ERR_INVALID_ARG;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!aligned16(target_shard) || !aligned16(gathered)) return UBT_ERR_INVALID_ARG;
  if (N > kMaxN) return UBT_ERR_UNSUPPORTED;
  if (B > 0 && (!workspace || !aligned16(workspace) ||
                workspace_bytes < verify_workspace_bytes((int64_t)B * N, Vs, UBT_VERIFY_SAMPLE)))
    return UBT_ERR_WORKSPACE;
  return UBT_OK;
}

int ubt_sample_totals_shard(const void* target_shard, int dtype, int B, int N, int Vs,
                            const unsigned long long* gathered_keys, int shards, float temperature,
                            unsigned long long* totals, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  const int rc = check_sample_shard(target_shard, dtype, B, N, Vs, gathered_keys, shards, workspace, workspace_bytes);
  if (rc != UBT_OK) return rc;
  if (!totals || !(temperature > 0.f)) return UBT_ERR_INVALID_ARG;
  if (B == 0) return UBT_OK;
  const int64_t rows = (int64_t)B * N;
  const VerifyWorkspace w = carve_verify_workspace(workspace, rows, Vs, UBT_VERIFY_SAMPLE);
  if (launch_row_totals_shard(target_shard, dtype, rows, Vs, gathered_keys, shards, temperature, w, totals,
                              static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return UBT_ERR_CUDA;
  return UBT_OK;
}

int ubt_sample_picks_shard(const void* target_shard, int dtype, int B, int N, int Vs, int v0, int rank,
                           const unsigned long long* gathered_totals, int shards, uint64_t seed, int32_t* picks,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
  const int rc = check_sample_shard(target_shard, dtype, B, N, Vs, gathered_totals, shards, workspace, workspace_bytes);
  if (rc != UBT_OK) return rc;
  if (!picks || v0 < 0 || rank < 0 || rank >= shards) return UBT_ERR_INVALID_ARG;
  if ((int64_t)v0 + Vs > 0x7fffffffll) return UBT_ERR_UNSUPPORTED;
  if (B == 0) return UBT_OK;
  const int64_t rows = (int64_t)B * N;
  const VerifyWorkspace w = carve_verify_workspace(workspace, rows, Vs, UBT_VERIFY_SAMPLE);
  if (launch_row_pick_shard(target_shard, dtype, rows, N, Vs, v0, rank, shards, gathered_totals, seed, w, picks,
                            static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return UBT_ERR_CUDA;
  return UBT_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------- host-buffer forms
namespace {
struct Carver {
  unsigned char* base;
  size_t off = 0;
  template <typename T> T* take(size_t count) {
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += align_up(count * sizeof(T), 256);
    return p;
  }
};

struct DeviceTree {
  ubt_tree t;
  void carve(Carver& c, int B, int L, int k, int N, bool cands) {
    t.B = B; t.N = N; t.L = L; t.k = k; t.mask_words = (N + 31) / 32;
    const size_t bn = (size_t)B * N;
    t.token_ids = c.take<int32_t>(bn); t.parents = c.take<int32_t>(bn); t.depths = c.take<int32_t>(bn);
    t.position_ids = c.take<int32_t>(bn); t.cand_rank = c.take<int32_t>(bn); t.scores = c.take<float>(bn);
    t.mask = c.take<uint32_t>(bn * t.mask_words); t.n_nodes = c.take<int32_t>((size_t)B);
    t.cand_ids = cands ? c.take<int32_t>((size_t)B * L * k) : nullptr;
    t.cand_logprob = cands ? c.take<float>((size_t)B * L * k) : nullptr;
  }
};

struct DraftHostLayout {
  void* logits; float* bigram; float *alpha, *lambda, *anchor_bigram; int32_t *anchor_tokens, *pos_offset, *status;
  DeviceTree tree; void* ws; size_t ws_bytes; size_t total;
  DraftHostLayout(void* buf, int B, int L, int V, int k, int N, int dtype) {
    Carver c{static_cast<unsigned char*>(buf)};
    logits = c.take<unsigned char>((size_t)B * L * V * esize(dtype));
    bigram = c.take<float>((size_t)B * (L - 1) * k * k);
    alpha = c.take<float>((size_t)L); lambda = c.take<float>((size_t)L);
    anchor_bigram = c.take<float>((size_t)B * k);
    anchor_tokens = c.take<int32_t>((size_t)B); pos_offset = c.take<int32_t>((size_t)B);
    status = c.take<int32_t>((size_t)B);
    tree.carve(c, B, L, k, N, true);
    ws_bytes = ubt_draft_workspace_bytes(B, L, V, k, N);
    ws = c.take<unsigned char>(ws_bytes);
    total = c.off;
  }
};

struct VerifyHostLayout {
  void* logits; DeviceTree tree; int32_t *accepted_len, *bonus, *accepted_nodes, *out_tokens, *node_pick, *status;
  void* ws; size_t ws_bytes; size_t total;
  VerifyHostLayout(void* buf, int B, int L, int N, int V, int dtype, int mode) {
    Carver c{static_cast<unsigned char*>(buf)};
    logits = c.take<unsigned char>((size_t)B * N * V * esize(dtype));
    tree.carve(c, B, L, 1, N, false);
    accepted_len = c.take<int32_t>((size_t)B); bonus = c.take<int32_t>((size_t)B);
    accepted_nodes = c.take<int32_t>((size_t)B * (L + 1)); out_tokens = c.take<int32_t>((size_t)B * (L + 1));
    node_pick = c.take<int32_t>((size_t)B * N);
    status = c.take<int32_t>((size_t)B);
    ws_bytes = ubt_verify_workspace_bytes(B, N, V, mode);
    ws = c.take<unsigned char>(ws_bytes);
    total = c.off;
  }
};

#define UBT_CUDA_OK(call) do { if ((call) != cudaSuccess) { cudaGetLastError(); return UBT_ERR_CUDA; } } while (0)

// End of a host-buffer call: copy the status words back if anybody wants them, wait for the stream, and turn
// flagged sequences into a return code when the caller asked for validation.
int finish_host_call(cudaStream_t st, const int32_t* dev_status, int32_t* host_status, bool validate, int B) {
  int32_t local[64];
  int32_t* dst = host_status;
  int32_t* heap = nullptr;
  if (!dst && validate) dst = B <= 64 ? local : (heap = new (std::nothrow) int32_t[(size_t)B]);
  if ((host_status || validate) && !dst) return UBT_ERR_CUDA;
  int rc = UBT_OK;
  if (dst && cudaMemcpyAsync(dst, dev_status, sizeof(int32_t) * (size_t)B, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    rc = UBT_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) rc = UBT_ERR_CUDA;
  if (rc == UBT_OK && validate) {
    int bits = 0;
    for (int b = 0; b < B; ++b) bits |= dst[b];
    if (bits & UBT_STATUS_WAIT_GAVE_UP) rc = UBT_ERR_CUDA;
    else if (bits & UBT_STATUS_NONFINITE) rc = UBT_ERR_NONFINITE;
  }
  delete[] heap;
  if (rc != UBT_OK) cudaGetLastError();
  return rc;
}
}  // namespace

extern "C" {

size_t ubt_draft_host_buffer_bytes(int B, int L, int V, int k, int N, int dtype) {
  if (check_shape(B, L, V, k, N) != UBT_OK || (dtype != UBT_F32 && dtype != UBT_BF16)) return 0;
  return DraftHostLayout(nullptr, B, L, V, k, N, dtype).total;
}

size_t ubt_verify_host_buffer_bytes(int B, int L, int N, int V, int dtype, int mode) {
  if (B < 0 || L < 1 || N < 1 || V < 1 || (dtype != UBT_F32 && dtype != UBT_BF16)) return 0;
  if (mode != UBT_VERIFY_GREEDY && mode != UBT_VERIFY_SAMPLE) return 0;
  return VerifyHostLayout(nullptr, B, L, N, V, dtype, mode).total;
}

int ubt_draft_tree_host(const void* unigram_logits, int dtype, const float* bigram_scores, int B, int L, int V, int k,
                        int N, const ubt_draft_opts* opts, ubt_tree* out, void* device_buffer,
                        size_t device_buffer_bytes, void* cuda_stream) {
  int rc = check_shape(B, L, V, k, N);
  if (rc) return rc;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!unigram_logits || !out || (L > 1 && !bigram_scores)) return UBT_ERR_INVALID_ARG;
  if (out->B != B || out->N != N || out->L != L || out->k != k) return UBT_ERR_INVALID_ARG;
  if ((rc = check_draft_opts(opts))) return rc;
  if (!device_buffer || !aligned16(device_buffer) ||
      device_buffer_bytes < ubt_draft_host_buffer_bytes(B, L, V, k, N, dtype))
    return UBT_ERR_WORKSPACE;
  if (B == 0) return UBT_OK;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  DraftHostLayout d(device_buffer, B, L, V, k, N, dtype);
  UBT_CUDA_OK(cudaMemcpyAsync(d.logits, unigram_logits, (size_t)B * L * V * esize(dtype), cudaMemcpyHostToDevice, st));
  if (L > 1)
    UBT_CUDA_OK(cudaMemcpyAsync(d.bigram, bigram_scores, sizeof(float) * (size_t)B * (L - 1) * k * k,
                                cudaMemcpyHostToDevice, st));
  ubt_draft_opts dev_opts{};
  if (opts) {
    dev_opts.search_width = opts->search_width;
    dev_opts.depth_bonus = opts->depth_bonus;
    if (opts->alpha) { UBT_CUDA_OK(cudaMemcpyAsync(d.alpha, opts->alpha, sizeof(float) * L, cudaMemcpyHostToDevice, st)); dev_opts.alpha = d.alpha; }
    if (opts->lambda) { UBT_CUDA_OK(cudaMemcpyAsync(d.lambda, opts->lambda, sizeof(float) * L, cudaMemcpyHostToDevice, st)); dev_opts.lambda = d.lambda; }
    if (opts->anchor_bigram) { UBT_CUDA_OK(cudaMemcpyAsync(d.anchor_bigram, opts->anchor_bigram, sizeof(float) * (size_t)B * k, cudaMemcpyHostToDevice, st)); dev_opts.anchor_bigram = d.anchor_bigram; }
    if (opts->anchor_tokens) { UBT_CUDA_OK(cudaMemcpyAsync(d.anchor_tokens, opts->anchor_tokens, sizeof(int32_t) * B, cudaMemcpyHostToDevice, st)); dev_opts.anchor_tokens = d.anchor_tokens; }
    if (opts->pos_offset) { UBT_CUDA_OK(cudaMemcpyAsync(d.pos_offset, opts->pos_offset, sizeof(int32_t) * B, cudaMemcpyHostToDevice, st)); dev_opts.pos_offset = d.pos_offset; }
    dev_opts.event_between = opts->event_between;
  }
  int32_t* host_status = opts ? opts->status : nullptr;  // a HOST array in this form
  const bool validate = opts && opts->validate_finite;
  dev_opts.status = (host_status || validate) ? d.status : nullptr;
  rc = ubt_draft_tree(d.logits, dtype, L > 1 ? d.bigram : nullptr, B, L, V, k, N, &dev_opts, &d.tree.t, d.ws,
                      d.ws_bytes, cuda_stream);
  if (rc) return rc;
  const size_t bn = (size_t)B * N;
  const ubt_tree& t = d.tree.t;
  struct { void* dst; const void* src; size_t bytes; } copies[] = {
      {out->token_ids, t.token_ids, bn * 4}, {out->parents, t.parents, bn * 4}, {out->depths, t.depths, bn * 4},
      {out->position_ids, t.position_ids, bn * 4}, {out->cand_rank, t.cand_rank, bn * 4},
      {out->scores, t.scores, bn * 4}, {out->mask, t.mask, bn * t.mask_words * 4}, {out->n_nodes, t.n_nodes, (size_t)B * 4},
      {out->cand_ids, t.cand_ids, (size_t)B * L * k * 4}, {out->cand_logprob, t.cand_logprob, (size_t)B * L * k * 4}};
  for (auto& c : copies)
    if (c.dst) UBT_CUDA_OK(cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyDeviceToHost, st));
  return finish_host_call(st, d.status, host_status, validate, B);
}

int ubt_verify_tree_host(const ubt_tree* tree, const void* target_logits, int dtype, int V, int mode,
                         const ubt_verify_opts* opts, ubt_verify_result* out, void* device_buffer,
                         size_t device_buffer_bytes, void* cuda_stream) {
  if (!tree || !target_logits || !out || V < 1) return UBT_ERR_INVALID_ARG;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (mode != UBT_VERIFY_GREEDY && mode != UBT_VERIFY_SAMPLE) return UBT_ERR_INVALID_ARG;
  const int B = tree->B, N = tree->N, L = tree->L;
  if (B < 0 || N < 1 || L < 1) return UBT_ERR_INVALID_ARG;
  if (N > kMaxN || L > kMaxL) return UBT_ERR_UNSUPPORTED;
  if (!tree->token_ids || !tree->parents || !tree->n_nodes) return UBT_ERR_INVALID_ARG;
  if (!out->accepted_len || !out->bonus_token || !out->accepted_nodes || !out->out_tokens) return UBT_ERR_INVALID_ARG;
  if (!device_buffer || !aligned16(device_buffer) ||
      device_buffer_bytes < ubt_verify_host_buffer_bytes(B, L, N, V, dtype, mode))
    return UBT_ERR_WORKSPACE;
  if (B == 0) return UBT_OK;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VerifyHostLayout d(device_buffer, B, L, N, V, dtype, mode);
  const size_t bn = (size_t)B * N;
  UBT_CUDA_OK(cudaMemcpyAsync(d.logits, target_logits, bn * V * esize(dtype), cudaMemcpyHostToDevice, st));
  UBT_CUDA_OK(cudaMemcpyAsync(d.tree.t.token_ids, tree->token_ids, bn * 4, cudaMemcpyHostToDevice, st));
  UBT_CUDA_OK(cudaMemcpyAsync(d.tree.t.parents, tree->parents, bn * 4, cudaMemcpyHostToDevice, st));
  UBT_CUDA_OK(cudaMemcpyAsync(d.tree.t.n_nodes, tree->n_nodes, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  ubt_verify_opts dev_opts{0, 1.0f, nullptr, nullptr, nullptr, 0, nullptr, 0, 0};
  if (opts) { dev_opts = *opts; }
  dev_opts.early_start = 0;  // the logits are copied in just before: nothing to start ahead of
  int32_t* host_status = dev_opts.status;  // a HOST array in this form
  const bool validate = dev_opts.validate_finite != 0;
  dev_opts.status = (host_status || validate) ? d.status : nullptr;
  int32_t* host_pick = dev_opts.node_pick;
  dev_opts.node_pick = host_pick ? d.node_pick : nullptr;
  ubt_verify_result r{d.accepted_len, d.bonus, d.accepted_nodes, d.out_tokens};
  int rc = ubt_verify_tree(&d.tree.t, d.logits, dtype, V, mode, &dev_opts, &r, d.ws, d.ws_bytes, cuda_stream);
  if (rc) return rc;
  UBT_CUDA_OK(cudaMemcpyAsync(out->accepted_len, d.accepted_len, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
  UBT_CUDA_OK(cudaMemcpyAsync(out->bonus_token, d.bonus, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
  UBT_CUDA_OK(cudaMemcpyAsync(out->accepted_nodes, d.accepted_nodes, (size_t)B * (L + 1) * 4, cudaMemcpyDeviceToHost, st));
  UBT_CUDA_OK(cudaMemcpyAsync(out->out_tokens, d.out_tokens, (size_t)B * (L + 1) * 4, cudaMemcpyDeviceToHost, st));
  if (host_pick) UBT_CUDA_OK(cudaMemcpyAsync(host_pick, d.node_pick, bn * 4, cudaMemcpyDeviceToHost, st));
  return finish_host_call(st, d.status, host_status, validate, B);
}

}  // extern "C"
namespace ubt {
cudaError_t ring_timeouts_verify(unsigned int* out);
cudaError_t ring_timeouts_topk(unsigned int* out);
cudaError_t ring_timeouts_path(unsigned int* out);
cudaError_t lm_head_timeouts(unsigned int* out);
}  // namespace ubt
extern "C" {
long long ubt_debug_ring_timeouts(void) {
  unsigned int a = 0, b = 0, c = 0, d = 0, e = 0;
  if (ring_timeouts_verify(&a) != cudaSuccess || ring_timeouts_topk(&b) != cudaSuccess ||
      ring_timeouts_path(&c) != cudaSuccess || lm_head_timeouts(&d) != cudaSuccess ||
      selector_timeouts(&e) != cudaSuccess)
    return -1;
  return (long long)a + b + c + d + e;
}

#ifdef UBT_BOUNDS_CHECK
}  // extern "C"
namespace ubt {
cudaError_t bounds_report_topk(long long out[4]);
cudaError_t bounds_report_tree(long long out[4]);
cudaError_t bounds_report_verify(long long out[4]);
}  // namespace ubt
extern "C" {
// Debug builds only (-DUBT_BOUNDS_CHECK): which = 0 top-k, 1 tree, 2 verify; out = flag, site, index, limit.
int ubt_debug_bounds_report(int which, long long out[4]) {
  cudaError_t e = which == 0 ? bounds_report_topk(out) : which == 1 ? bounds_report_tree(out) : bounds_report_verify(out);
  return e == cudaSuccess ? UBT_OK : UBT_ERR_CUDA;
}
#endif

int ubt_verify_keys_shard(const void* target_shard, int dtype, int B, int N, int Vs, int v0,
                          unsigned long long* row_keys, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!target_shard || !row_keys || B < 0 || N < 1 || Vs < 1 || v0 < 0) return UBT_ERR_INVALID_ARG;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!aligned16(target_shard) || !aligned16(row_keys)) return UBT_ERR_INVALID_ARG;
  if (N > kMaxN || (int64_t)v0 + Vs > 0x7fffffffll) return UBT_ERR_UNSUPPORTED;
  if (B == 0) return UBT_OK;
  const int64_t rows = (int64_t)B * N;
  if (!workspace || !aligned16(workspace) || workspace_bytes < verify_workspace_bytes(rows, Vs, UBT_VERIFY_GREEDY))
    return UBT_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  VerifyWorkspace w = carve_verify_workspace(workspace, rows, Vs, UBT_VERIFY_GREEDY);
  if (launch_row_argmax(target_shard, dtype, rows, Vs, w, 0, false, st) != cudaSuccess) return UBT_ERR_CUDA;
  if (launch_row_keys_shard(w, rows, Vs, v0, row_keys, st) != cudaSuccess) return UBT_ERR_CUDA;
  return UBT_OK;
}

int ubt_verify_tree_keys(const ubt_tree* tree, const unsigned long long* gathered_keys, int shards,
                         ubt_verify_result* out, const ubt_verify_opts* opts, void* cuda_stream) {
  if (!tree || !out || !gathered_keys || shards < 1) return UBT_ERR_INVALID_ARG;
  if (!tree->token_ids || !tree->parents || !tree->n_nodes) return UBT_ERR_INVALID_ARG;
  if (!out->accepted_len || !out->bonus_token || !out->accepted_nodes || !out->out_tokens) return UBT_ERR_INVALID_ARG;
  if (!aligned16(gathered_keys)) return UBT_ERR_INVALID_ARG;
  const int B = tree->B, N = tree->N, L = tree->L;
  if (B < 0 || N < 1 || L < 1) return UBT_ERR_INVALID_ARG;
  if (N > kMaxN || L > kMaxL) return UBT_ERR_UNSUPPORTED;
  if (B == 0) return UBT_OK;
  if (launch_walk_keys(*tree, gathered_keys, shards, opts ? opts->node_pick : nullptr, *out,
                       opts ? opts->status : nullptr, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return UBT_ERR_CUDA;
  return UBT_OK;
}

}  // extern "C"
