// Merge of the per-segment partials of step a1 into a row's candidates (one warp per row).
// Used by the standalone merge kernel and by the prologue of the tree kernel.
#pragma once

#include "ubt_common.cuh"

namespace ubt {

// The partial arrays the streaming kernel wrote (see TopkWorkspace); parts.part_ms == nullptr means "none".
struct MergeParts {
  SpanPlan plan;
  const float* part_ms;     // [rows, smax, 2]  (max, sum of exp relative to it)
  const float* part_val;    // [rows, smax, k]
  const int32_t* part_idx;  // [rows, smax, k]
  const int32_t* part_cnt;  // [rows, smax]
};

// Status bits of a sequence (ubt_draft_opts.status / ubt_verify_opts.status).
constexpr int kStatusNonFinite = 1;  // a NaN or +inf among the logits
constexpr int kStatusWaitGaveUp = 2; // a bounded device-side wait gave up: results undefined

// Every lane of one warp calls this for the same row; returns the row's status bits (all lanes agree): the
// log-sum-exp of a row that holds a NaN or +inf is not finite, and a segment whose streaming CTA gave up a wait
// carries the count -1.  Writes cand_ids[row, 0..k) (best first) and
// cand_lp[row, r] = value - log-sum-exp of the whole row; sm_ids / sm_lp, if given, receive a copy of the row's k
// entries (the caller's shared-memory staging).
__device__ __forceinline__ int merge_row_warp(const MergeParts& p, int64_t rows, int64_t row, int V, int k,
                                               int32_t* __restrict__ cand_ids_, float* __restrict__ cand_lp_,
                                               int lane, int* sm_ids = nullptr, float* sm_lp = nullptr) {
  const long long nslots = rows * p.plan.smax;
  const Span<const float> part_ms(p.part_ms, nslots * 2, 321), part_val(p.part_val, nslots * k, 322);
  const Span<const int32_t> part_idx(p.part_idx, nslots * k, 323), part_cnt(p.part_cnt, nslots, 324);
  const Span<int32_t> cand_ids(cand_ids_, rows * k, 325);
  const Span<float> cand_lp(cand_lp_, rows * k, 326);
  const int64_t c_first = (row * (int64_t)V) / p.plan.span;
  const int64_t c_last = ((row + 1) * (int64_t)V - 1) / p.plan.span;
  const int nseg = (int)(c_last - c_first + 1);
  const int64_t base = row * p.plan.smax;

  // every global load of the common case is issued before anything depends on one: a single round trip
  const int nq = nseg * k;
  float my_m = -1.0e30f, my_s = 0.f;
  if (lane < nseg) { my_m = part_ms[(base + lane) * 2]; my_s = part_ms[(base + lane) * 2 + 1]; }
  uint64_t key[2] = {0ull, 0ull};
  float val[2] = {0.f, 0.f};
  int pidx[2] = {0, 0}, pcnt[2] = {0, 0}, pi[2] = {0, 0};
  if (nq <= 64) {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int q = lane + 32 * c;
      const int j = q / k, i = q - j * k;
      pi[c] = i;
      if (q < nq) {
        pcnt[c] = part_cnt[base + j];  // -1: the CTA of this segment gave up (no entry passes the mask below)
        val[c] = part_val[(base + j) * k + i];   // slots beyond the count hold stale data: masked below
        pidx[c] = part_idx[(base + j) * k + i];
      }
    }
  }
  float M = my_m;
  for (int j = lane + 32; j < nseg; j += 32) M = fmaxf(M, part_ms[(base + j) * 2]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(FULL, M, o));
  float S = lane < nseg ? my_s * exp2f((my_m - M) * kLog2e) : 0.f;
  for (int j = lane + 32; j < nseg; j += 32)
    S += part_ms[(base + j) * 2 + 1] * exp2f((part_ms[(base + j) * 2] - M) * kLog2e);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(FULL, S, o);
  const float lse = M + logf(S);

  int found = 0;
  if (nq <= 64) {
    // The usual case (a row is cut into a few segments): every lane holds up to two entries in registers,
    // and the exact ranks are counted by exchanging keys with shuffles.
#pragma unroll
    for (int c = 0; c < 2; ++c)
      if (lane + 32 * c < nq && pi[c] < pcnt[c]) key[c] = make_key(val[c], pidx[c]);
    int rank[2] = {0, 0};
#pragma unroll
    for (int c2 = 0; c2 < 2; ++c2) {
      const int n2 = nq - 32 * c2 < 32 ? nq - 32 * c2 : 32;
      for (int l2 = 0; l2 < n2; ++l2) {
        const uint64_t other = __shfl_sync(FULL, key[c2], l2);
        rank[0] += other > key[0];
        rank[1] += other > key[1];
      }
    }
#pragma unroll
    for (int c = 0; c < 2; ++c)
      if (key[c] != 0ull && rank[c] < k) {
        cand_ids[row * k + rank[c]] = key_idx(key[c]);
        cand_lp[row * k + rank[c]] = val[c] - lse;
        if (sm_ids) { sm_ids[rank[c]] = key_idx(key[c]); sm_lp[rank[c]] = val[c] - lse; }
      }
  } else {
    // Many entries (large k, or a row cut into many segments): every segment's list is sorted best first, so an
    // entry's rank is its place in its own list plus, per other segment, the number of better keys there,
    // found by binary search.
    for (int q = lane; q < nq; q += 32) {
      const int j = q / k, i = q - j * k;
      if (i >= part_cnt[base + j]) continue;  // also skips a segment that gave up (count -1)
      const float val = part_val[(base + j) * k + i];
      const int idx = part_idx[(base + j) * k + i];
      const uint64_t key = make_key(val, idx);
      int rank = i;
      for (int j2 = 0; j2 < nseg && rank < k; ++j2) {
        if (j2 == j) continue;
        int lo = 0, hi = part_cnt[base + j2];  // list[0..lo) > key, list[hi..) < key
        hi = hi < 0 ? 0 : hi;
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (make_key(part_val[(base + j2) * k + mid], part_idx[(base + j2) * k + mid]) > key) lo = mid + 1;
          else hi = mid;
        }
        rank += lo;
      }
      if (rank < k) {
        cand_ids[row * k + rank] = idx;
        cand_lp[row * k + rank] = val - lse;
        if (sm_ids) { sm_ids[rank] = idx; sm_lp[rank] = val - lse; }
      }
    }
  }
  int gave_up = 0;
  for (int j = lane; j < nseg; j += 32) {
    const int c = part_cnt[base + j];
    gave_up |= c < 0;
    found += c < 0 ? 0 : c;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) found += __shfl_xor_sync(FULL, found, o);
  gave_up = __any_sync(FULL, gave_up);
  for (int r = found + lane; r < k; r += 32) {  // fewer than k entries above -inf: documented as unsupported
    cand_ids[row * k + r] = -1;
    cand_lp[row * k + r] = -INFINITY;
    if (sm_ids) { sm_ids[r] = -1; sm_lp[r] = -INFINITY; }
  }
  return ((lse == lse && lse < INFINITY) ? 0 : kStatusNonFinite) | (gave_up ? kStatusWaitGaveUp : 0);
}

// ---------------------------------------------------------------------------------------- one CTA per row
// The same merge by a whole CTA with the lists staged in shared memory, for rows with many entries (large k, many
// segments) and for the two ends of a vocabulary-parallel a1:
//   * source: the segment partials of this GPU's streaming kernel (`shards` == 0), or `shards` per-row partials
//     gathered from the ranks of a vocabulary-parallel group, rank r's arrays `shard_bytes` * r bytes behind rank
//     0's ([rows,2] (max, sum exp), [rows,k] values, [rows,k] token ids of the whole vocabulary, [rows] counts);
//   * result: the row's candidates (ids, value - log-sum-exp of the row), or, with MergeShardOut::ms set, this
//     rank's per-row partial in that format: raw values, ids moved by `id_offset` (the first column of the rank's
//     slice), (max, sum exp) and the count (-1 if a streaming CTA of the row gave up a wait).
struct MergeSource {
  MergeParts parts;
  int shards;
  int64_t shard_bytes;
};
struct MergeShardOut {
  float* ms;
  float* val;
  int32_t* idx;
  int32_t* cnt;
  int id_offset;
};

// s_key: [lists * k] keys, s_cnt: [lists], s_red: [2]; every thread of the CTA calls this for the same row.
template <int THREADS>
__device__ __forceinline__ void merge_row_cta(const MergeSource& src, int64_t rows, int64_t row, int V, int k,
                                              int32_t* __restrict__ cand_ids, float* __restrict__ cand_lp,
                                              const MergeShardOut& so, unsigned long long* s_key, int* s_cnt,
                                              float* s_red) {
  const MergeParts& p = src.parts;
  const int tid = threadIdx.x, lane = tid & 31;
  int nseg;
  int64_t base = 0;
  if (src.shards) {
    nseg = src.shards;
  } else {
    const int64_t c_first = (row * (int64_t)V) / p.plan.span;
    const int64_t c_last = ((row + 1) * (int64_t)V - 1) / p.plan.span;
    nseg = (int)(c_last - c_first + 1);
    base = row * p.plan.smax;
  }
  auto shard = [&](const void* a, int j) { return static_cast<const char*>(a) + (int64_t)j * src.shard_bytes; };
  auto ms_of = [&](int j) {
    return src.shards ? reinterpret_cast<const float*>(shard(p.part_ms, j)) + row * 2 : p.part_ms + (base + j) * 2;
  };
  auto val_of = [&](int j) {
    return src.shards ? reinterpret_cast<const float*>(shard(p.part_val, j)) + row * k : p.part_val + (base + j) * k;
  };
  auto idx_of = [&](int j) {
    return src.shards ? reinterpret_cast<const int32_t*>(shard(p.part_idx, j)) + row * k : p.part_idx + (base + j) * k;
  };
  auto cnt_of = [&](int j) {
    return src.shards ? reinterpret_cast<const int32_t*>(shard(p.part_cnt, j))[row] : p.part_cnt[base + j];
  };

  for (int j = tid; j < nseg; j += THREADS) s_cnt[j] = cnt_of(j);
  __syncthreads();
  const int nq = nseg * k;
  for (int q = tid; q < nq; q += THREADS) {
    const int j = q / k, i = q - j * k;
    s_key[q] = i < s_cnt[j] ? make_key(val_of(j)[i], idx_of(j)[i]) : 0ull;  // slots beyond the count hold stale data
  }
  if (tid < 32) {
    float M = -1.0e30f;
    for (int j = lane; j < nseg; j += 32) M = fmaxf(M, ms_of(j)[0]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(FULL, M, o));
    float S = 0.f;
    for (int j = lane; j < nseg; j += 32) S += ms_of(j)[1] * exp2f((ms_of(j)[0] - M) * kLog2e);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) S += __shfl_xor_sync(FULL, S, o);
    if (lane == 0) { s_red[0] = M; s_red[1] = S; }
  }
  __syncthreads();
  const float M = s_red[0], S = s_red[1];
  const float sub = so.ms ? 0.f : M + logf(S);
  int32_t* ids_out = so.ms ? so.idx : cand_ids;
  float* val_out = so.ms ? so.val : cand_lp;
  // every list is sorted best first: an entry's rank is its place in its own list plus, per other list, the
  // number of better keys there (binary search); keys are unique, so ranks are
  for (int q = tid; q < nq; q += THREADS) {
    const unsigned long long key = s_key[q];
    if (key == 0ull) continue;
    const int j = q / k;
    int rank = q - j * k;
    for (int j2 = 0; j2 < nseg && rank < k; ++j2) {
      if (j2 == j) continue;
      int lo = 0, hi = s_cnt[j2] < 0 ? 0 : s_cnt[j2];  // list[0..lo) > key, list[hi..) < key
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (s_key[j2 * k + mid] > key) lo = mid + 1;
        else hi = mid;
      }
      rank += lo;
    }
    if (rank < k) {
      ids_out[row * k + rank] = key_idx(key) + so.id_offset;
      val_out[row * k + rank] = key_val(key) - sub;
    }
  }
  int found = 0, gave_up = 0;
  for (int j = 0; j < nseg; ++j) {
    gave_up |= s_cnt[j] < 0;
    found += s_cnt[j] < 0 ? 0 : s_cnt[j];
  }
  for (int r = found + tid; r < k; r += THREADS) {  // fewer than k entries in the whole row
    ids_out[row * k + r] = -1;
    val_out[row * k + r] = -INFINITY;
  }
  if (so.ms && tid == 0) {
    so.ms[row * 2] = M;
    so.ms[row * 2 + 1] = S;
    so.cnt[row] = gave_up ? -1 : (found < k ? found : k);
  }
}

}  // namespace ubt
