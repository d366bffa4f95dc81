// Launchers shared between the translation units of libubt (host side, not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <atomic>
#include <stddef.h>
#include <stdint.h>

#include "../../include/ubt.h"
#include "ubt_common.cuh"
#include "ubt_merge.cuh"

namespace ubt {

constexpr int kMaxK = 64;
constexpr int kMaxN = 256;
constexpr int kMaxL = 64;
constexpr size_t kTreeTableBytes = 160 * 1024;

// Kernel launch with or without programmatic dependent launch (see pdl_wait in ubt_common.cuh).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                 bool programmatic, Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = programmatic ? attr : nullptr;
  cfg.numAttrs = programmatic ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

struct DeviceInfo {
  int device;
  int sm_count;
  int max_smem_optin;
};
// Properties of the current device (queried once per device, cached).
const DeviceInfo& device_info();

// Lets kernel `Kern` use up to the device's opt-in maximum of dynamic shared memory.  The attribute belongs to
// the (function, device) pair, so it is set once per device and per kernel instantiation, with that device current.
template <auto Kern>
inline cudaError_t allow_max_dynamic_smem() {
  static std::atomic<bool> done[64];
  const DeviceInfo& di = device_info();
  const int dev = di.device;
  if (done[dev].load(std::memory_order_acquire)) return cudaSuccess;
  cudaFuncAttributes fa{};
  cudaError_t e = cudaFuncGetAttributes(&fa, Kern);
  if (e != cudaSuccess) return e;
  // the limit covers static and dynamic shared memory together
  e = cudaFuncSetAttribute(Kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           di.max_smem_optin - (int)fa.sharedSizeBytes);
  if (e == cudaSuccess) done[dev].store(true, std::memory_order_release);
  return e;
}

// Cut rows*V elements into equal contiguous spans, one per CTA.
SpanPlan make_span_plan(int64_t rows, int V, int ctas, int64_t min_span);

// ---- a1: per-row (max, sum-exp, top-k) partials, then the per-row merge --------------------
struct TopkWorkspace {
  SpanPlan plan;
  float* part_ms;     // [rows, smax, 2]
  float* part_val;    // [rows, smax, k]
  int32_t* part_idx;  // [rows, smax, k]
  int32_t* part_cnt;  // [rows, smax]
};
SpanPlan topk_plan(int64_t rows, int V);
size_t topk_workspace_bytes(int64_t rows, int V, int k);
TopkWorkspace carve_topk_workspace(void* ws, int64_t rows, int V, int k);
cudaError_t launch_lse_topk(const void* logits, int dtype, int64_t rows, int V, int k,
                            const TopkWorkspace& w, cudaStream_t st);
cudaError_t launch_merge_topk(int64_t rows, int V, int k, const TopkWorkspace& w, int32_t* cand_ids,
                              float* cand_lp, cudaStream_t st);
// Vocabulary-parallel a1: this rank's per-row partial from its slice, and the merge of the gathered partials.
size_t shard_partial_bytes(int64_t rows, int k);
// The four arrays of one rank's partial inside its buffer, ids to be moved by id_offset when written.
MergeShardOut carve_shard_partial(void* partial, int64_t rows, int k, int id_offset);
cudaError_t launch_merge_topk_shard(int64_t rows, int V, int k, const TopkWorkspace& w, void* partial, int v0,
                                    cudaStream_t st);
cudaError_t launch_merge_shards(const void* gathered, int shards, int64_t rows, int k, int32_t* cand_ids,
                                float* cand_lp, cudaStream_t st);
inline MergeParts merge_parts(const TopkWorkspace& w) {
  return MergeParts{w.plan, w.part_ms, w.part_val, w.part_idx, w.part_cnt};
}
inline MergeParts no_merge_parts() { return MergeParts{SpanPlan{0, 0, 0}, nullptr, nullptr, nullptr, nullptr}; }

// ---- selector scores (between a1 and a2)
constexpr int kMaxSelectorRank = 8192;
cudaError_t launch_selector_scores(const void* phi, const void* psi, int dtype, int V, int R, const float* gate,
                                   const int32_t* cand_ids, const int32_t* anchor_tokens, int B, int L, int k,
                                   float* bigram, float* anchor_bigram, cudaStream_t st);

// ---- a2 + a3 + a3b --------------------------------------------------------------------------
size_t tree_smem_bytes(int L, int k, int N);
// `parts` with a non-null part_ms makes the kernel merge the step-a1 partials itself (V is then the row
// length they were cut from) and write out.cand_ids / out.cand_logprob; otherwise it reads them.
cudaError_t launch_build_tree(const float* bigram, int B, int L, int k, int N, int W, float zeta,
                              const float* alpha, const float* lambda, const float* anchor_bigram,
                              const int32_t* anchor_tokens, const int32_t* pos_offset,
                              const ubt_tree& out, const MergeParts& parts, int V, int32_t* status, cudaStream_t st);
cudaError_t launch_build_mask(const ubt_tree& tree, const int32_t* pos_offset, cudaStream_t st);

// ---- a4 ---------------------------------------------------------------------------------------
struct VerifyWorkspace {
  SpanPlan plan;                 // greedy: spans of the row-argmax kernel
  unsigned long long* part_key;  // greedy: [B*N, smax] (value, ~token) keys
  int32_t* pick;                 // sampling: [B*N] picks when the caller gave no node_pick
  float* row_ac;                 // sampling: [B*N, 2] per-row constants (a, c) of the weight routine
  unsigned long long* block_sum; // sampling: [B*N, nblocks] sums of the integer weights per 1024 tokens
  int nblocks;
};
size_t verify_workspace_bytes(int64_t rows, int V, int mode);
VerifyWorkspace carve_verify_workspace(void* ws, int64_t rows, int V, int mode);
// neighbour_smem: dynamic shared memory of one CTA of the kernel launched just before on the stream (the tree
// kernel when draft and verify calls follow one another); the ring is sized to fit beside it on an SM.
// early: the kernel may start before the kernel in front of it on the stream has completed (programmatic
// dependent launch); the caller has checked that nothing it writes is still in use there.
cudaError_t launch_row_argmax(const void* logits, int dtype, int64_t rows, int V,
                              const VerifyWorkspace& w, size_t neighbour_smem, bool early, cudaStream_t st);
cudaError_t launch_row_sample(const void* logits, int dtype, int B, int N, int V, uint64_t seed,
                              float temperature, int32_t* pick, const VerifyWorkspace& w, bool early,
                              cudaStream_t st);
cudaError_t launch_walk(const ubt_tree& tree, int mode, const VerifyWorkspace& w, int V,
                        const int32_t* sampled_pick, int32_t* node_pick,
                        const ubt_verify_result& out, int32_t* status, cudaStream_t st, int pick_shards = 1);
// sampling a4 over a vocabulary-parallel group (see ubt_verify.cu)
cudaError_t launch_row_totals_shard(const void* logits, int dtype, int64_t rows, int Vs,
                                    const unsigned long long* gathered_keys, int shards, float temperature,
                                    const VerifyWorkspace& w, unsigned long long* totals, cudaStream_t st);
cudaError_t launch_row_pick_shard(const void* logits, int dtype, int64_t rows, int N, int Vs, int v0, int rank, int shards,
                                  const unsigned long long* gathered_totals, uint64_t seed, const VerifyWorkspace& w,
                                  int32_t* pick, cudaStream_t st);

// vocabulary-parallel greedy a4: one key per row of this rank's slice; the walk on the gathered keys
cudaError_t launch_row_keys_shard(const VerifyWorkspace& w, int64_t rows, int V, int v0, unsigned long long* row_keys,
                                  cudaStream_t st);
cudaError_t launch_walk_keys(const ubt_tree& tree, const unsigned long long* gathered_keys, int shards,
                             int32_t* node_pick, const ubt_verify_result& out, int32_t* status, cudaStream_t st);

cudaError_t selector_timeouts(unsigned int* out);

// ---- LM head fused with a1 (ubt_lmhead.cu): tcgen05 GEMM whose epilogue keeps (max, sum exp, top-k) per row
int lm_head_max_k();
int lm_head_max_rows();
size_t lm_head_workspace_bytes(int64_t rows, int k);
// shard_partial != nullptr: `weight` is the slice [V, d] of a vocabulary-parallel head that starts at column v0 of
// the whole vocabulary, and the result is this rank's partial (ubt_topk_shard's format) instead of candidates
cudaError_t launch_lm_head_topk(const void* hidden, const void* weight, int64_t rows, int d, int V, int k,
                                int32_t* cand_ids, float* cand_lp, void* ws, cudaStream_t st,
                                void* shard_partial = nullptr, int v0 = 0);

// ---- a4, path-only form: evaluates only the target rows the walk visits (ubt_verify_path.cu)
size_t verify_path_workspace_bytes(int B, int N, int mode);
int verify_path_max_batch();
cudaError_t launch_verify_path(const ubt_tree& tree, const void* logits, int dtype, int V, int mode, uint64_t seed,
                               float temperature, void* ws, int32_t* node_pick, const ubt_verify_result& out,
                               int32_t* status, cudaStream_t st);

}  // namespace ubt
