// Global merge: per query, the top-k of the n_part sorted partial lists, then the id gather.
// One CTA per query.  The lists are copied to shared memory; warp 0 then runs a k-round
// tournament over the list heads: each lane keeps the best head among the lists it owns and
// two warp max-reductions (score word, then slot word) pick the winner of the round.
#include <math.h>

#include "common.cuh"
#include "kernels.h"
#include "pipeline.cuh"

namespace icc {

constexpr int MERGE_THREADS = 256;

// Same tournament for any number of lists, with the list positions in shared memory.
__device__ __forceinline__ int tournament_in_shared(const uint64_t* cand, uint32_t* pos, int n_part, int k, int lane,
                                                    uint64_t* win_key) {
  uint64_t best = KEY_EMPTY;
  int best_p = -1;
  for (int p = lane; p < n_part; p += 32) {
    const uint64_t key = cand[(size_t)p * k];
    if (key > best) { best = key; best_p = p; }
  }
  int r = 0;
  for (; r < k; ++r) {
    const uint32_t hi = (uint32_t)(best >> 32);
    const uint32_t top_hi = __reduce_max_sync(FULL_MASK, hi);
    if (top_hi == 0) break;
    const uint32_t lo = (hi == top_hi) ? (uint32_t)best : 0u;
    const uint32_t top_lo = __reduce_max_sync(FULL_MASK, lo);
    if (hi == top_hi && lo == top_lo) {
      win_key[r] = best;
      pos[best_p] += 1;
      best = KEY_EMPTY;
      best_p = -1;
      for (int p = lane; p < n_part; p += 32) {
        const uint32_t j = pos[p];
        const uint64_t key = (j < (uint32_t)k) ? cand[(size_t)p * k + j] : KEY_EMPTY;
        if (key > best) { best = key; best_p = p; }
      }
    }
  }
  return r;
}

__global__ void __launch_bounds__(MERGE_THREADS)
merge_topk_kernel(const uint64_t* __restrict__ partials, int n_part, int nq, int k,
                  const int64_t* __restrict__ ids, int64_t* __restrict__ out_ids,
                  float* __restrict__ out_scores, uint64_t* __restrict__ out_keys,
                  uint64_t* __restrict__ out_thr, float min_score, int32_t* __restrict__ out_counts,
                  int64_t self_slot0) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t* cand = reinterpret_cast<uint64_t*>(smem_raw);                 // [n_part][k]
  uint32_t* pos = reinterpret_cast<uint32_t*>(cand + (size_t)n_part * k);  // [n_part]
  __shared__ uint64_t win_key[MAX_K];

  const int q = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
  const int total = n_part * k;
  grid_dep_launch_dependents();
  grid_dep_wait();   // the partial lists come from the previous kernel
  // list p of this query is k contiguous keys at partials[(p * nq + q) * k]; several loads
  // per thread are in flight at once
#pragma unroll 4
  for (int i = tid; i < total; i += MERGE_THREADS) {
    const int p = i / k, j = i - p * k;
    cand[i] = __ldg(partials + ((size_t)p * nq + q) * k + j);
  }
  for (int p = tid; p < n_part; p += MERGE_THREADS) pos[p] = 0;
  __syncthreads();

  if (tid < 32) {
    int r;
    if (n_part <= 32) r = tournament_in_registers<1>(cand, k, n_part, k, lane, win_key);
    else if (n_part <= 64) r = tournament_in_registers<2>(cand, k, n_part, k, lane, win_key);
    else if (n_part <= 96) r = tournament_in_registers<3>(cand, k, n_part, k, lane, win_key);
    else if (n_part <= 128) r = tournament_in_registers<4>(cand, k, n_part, k, lane, win_key);
    else if (n_part <= 160) r = tournament_in_registers<5>(cand, k, n_part, k, lane, win_key);
    else r = tournament_in_shared(cand, pos, n_part, k, lane, win_key);
    for (int i = r + lane; i < k; i += 32) win_key[i] = KEY_EMPTY;  // fewer than k candidates
  }
  __syncthreads();
  if (out_keys) {  // intermediate merge: keep the key form
    for (int i = tid; i < k; i += MERGE_THREADS) out_keys[(size_t)q * k + i] = win_key[i];
    if (tid == 0) out_thr[q] = win_key[k - 1];
    return;
  }
  if (self_slot0 >= 0) {
    // similarity to the OTHER entries: query q is cache row self_slot0 + q; report the best
    // entry that is not that row (one result per query)
    if (tid == 0) {
      uint64_t pick = KEY_EMPTY;
      for (int i = 0; i < k; ++i) {
        const uint64_t key = win_key[i];
        if (key != KEY_EMPTY && (int64_t)key_slot(key) != self_slot0 + q) {
          pick = key;
          break;
        }
      }
      out_scores[q] = (pick == KEY_EMPTY) ? -INFINITY : key_score(pick);
      out_ids[q] = (pick == KEY_EMPTY) ? (int64_t)-1 : ids[key_slot(pick)];
    }
    return;
  }
  // Entries below min_score (-inf = keep all) are reported as absent; the list is sorted, so
  // the kept entries are a prefix and their number is the query's hit count.
  int kept = 0;
  for (int i = tid; i < k; i += MERGE_THREADS) {
    const uint64_t key = win_key[i];
    const bool keep = (key != KEY_EMPTY) && (key_score(key) >= min_score);
    out_scores[(size_t)q * k + i] = keep ? key_score(key) : -INFINITY;
    out_ids[(size_t)q * k + i] = keep ? ids[key_slot(key)] : (int64_t)-1;
    kept += keep ? 1 : 0;
  }
  if (out_counts) {
    const int total_kept = __reduce_add_sync(FULL_MASK, kept);   // per warp
    __shared__ int warp_kept[MERGE_THREADS / 32];
    if (lane == 0) warp_kept[tid >> 5] = total_kept;
    __syncthreads();
    if (tid == 0) {
      int sum = 0;
      for (int w2 = 0; w2 < MERGE_THREADS / 32; ++w2) sum += warp_kept[w2];
      out_counts[q] = sum;
    }
  }
}

static int g_merge_smem_limit = 48 * 1024;

cudaError_t merge_configure(int smem_optin) {
  cudaError_t e = cudaFuncSetAttribute(merge_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       smem_optin - 2048);
  if (e == cudaSuccess) g_merge_smem_limit = smem_optin - 2048;
  return e;
}

cudaError_t launch_merge(const uint64_t* partials, int n_part, int nq, int k, const int64_t* ids,
                         int64_t* out_ids, float* out_scores, float min_score, int32_t* out_counts,
                         cudaStream_t st, int64_t self_slot0) {
  const size_t smem = (size_t)n_part * k * 8 + (size_t)n_part * 4;
  if (smem > (size_t)g_merge_smem_limit) return cudaErrorInvalidValue;
  return launch_overlapped(merge_topk_kernel, dim3(nq), dim3(MERGE_THREADS), smem, st, 1, partials, n_part, nq, k, ids,
                           out_ids, out_scores, (uint64_t*)nullptr, (uint64_t*)nullptr, min_score, out_counts,
                           self_slot0);
}

cudaError_t launch_merge_keys(const uint64_t* partials, int n_part, int nq, int k, uint64_t* out_keys,
                              uint64_t* out_thr, cudaStream_t st) {
  const size_t smem = (size_t)n_part * k * 8 + (size_t)n_part * 4;
  if (smem > (size_t)g_merge_smem_limit || !out_keys || !out_thr) return cudaErrorInvalidValue;
  return launch_overlapped(merge_topk_kernel, dim3(nq), dim3(MERGE_THREADS), smem, st, 1, partials, n_part, nq, k,
                           (const int64_t*)nullptr, (int64_t*)nullptr, (float*)nullptr, out_keys, out_thr, -INFINITY,
                           (int32_t*)nullptr, (int64_t)-1);
}

}  // namespace icc
