// Greedy verification without any caller-provided scratch.
//
// Some callers cannot allocate device memory at the point where they verify a tree: code running inside
// a memory pool that is already fully handed out, a plugin that is only given its input and output
// buffers, a real-time loop where cudaMalloc's implicit synchronisation is not acceptable.  For them this
// file keeps the row-key scratch of the greedy verification in a fixed array inside the library image.
#include <mutex>

#include "ubt_internal.h"

namespace ubt {

// 65,536 keys of 8 bytes = 512 KiB, resident on every GPU that loads the library until the process exits.
constexpr long long kStaticKeys = 65536;
static __device__ __align__(256) unsigned long long g_static_row_keys[kStaticKeys];

// Device address of the array on the CURRENT device.  In host code the array's name is only a stand-in for
// the symbol, not a device pointer, so the address is asked for once per device and cached.
static cudaError_t static_row_keys(unsigned long long** out) {
  static unsigned long long* addr[64];
  static bool known[64];
  static std::mutex mu;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_row_keys);
    if (e != cudaSuccess) return e;
    addr[dev] = static_cast<unsigned long long*>(p);
    known[dev] = true;
  }
  *out = addr[dev];
  return cudaSuccess;
}

}  // namespace ubt

using namespace ubt;

extern "C" int ubt_verify_tree_static(const ubt_tree* tree, const void* target_logits, int dtype, int V,
                                      int32_t* node_pick, ubt_verify_result* out, void* cuda_stream) {
  if (!tree || !target_logits || !out || V < 1) return UBT_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(target_logits) & 15u) != 0) return UBT_ERR_INVALID_ARG;
  if (dtype != UBT_F32 && dtype != UBT_BF16) return UBT_ERR_INVALID_ARG;
  if (!tree->token_ids || !tree->parents || !tree->n_nodes) return UBT_ERR_INVALID_ARG;
  if (!out->accepted_len || !out->bonus_token || !out->accepted_nodes || !out->out_tokens) return UBT_ERR_INVALID_ARG;
  const int B = tree->B, N = tree->N, L = tree->L;
  if (B < 0 || N < 1 || L < 1) return UBT_ERR_INVALID_ARG;
  if (N > kMaxN || L > kMaxL) return UBT_ERR_UNSUPPORTED;
  if (B == 0) return UBT_OK;
  const int64_t rows = (int64_t)B * N;
  // the span plan decides how many keys a row needs; nothing is written yet
  VerifyWorkspace w = carve_verify_workspace(nullptr, rows, V, UBT_VERIFY_GREEDY);
  if (rows * (int64_t)w.plan.smax > kStaticKeys) return UBT_ERR_STATIC_SCRATCH;
  unsigned long long* keys = nullptr;
  if (static_row_keys(&keys) != cudaSuccess) { cudaGetLastError(); return UBT_ERR_CUDA; }
  w.part_key = keys;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // plain stream order (no early start): the one shared array may still be read by the walk of a call in front
  if (launch_row_argmax(target_logits, dtype, rows, V, w, tree_smem_bytes(tree->L, tree->k, tree->N), false, st) !=
      cudaSuccess)
    return UBT_ERR_CUDA;
  if (launch_walk(*tree, UBT_VERIFY_GREEDY, w, V, nullptr, node_pick, *out, nullptr, st) != cudaSuccess) return UBT_ERR_CUDA;
  return UBT_OK;
}

extern "C" long long ubt_verify_static_capacity(void) { return kStaticKeys; }
