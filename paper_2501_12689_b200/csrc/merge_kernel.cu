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

constexpr int SELECT_THREADS = 256;
constexpr int SELECT_MAX_VALUES = 1280;

// Per query: the k-th largest of m = n_tiles * 4 group maxima, by rank counting (m is a few
// hundred).  CTA (q, c) ranks values c*256 .. c*256+255 of query q, one per thread, against a
// shared copy of all m values held as unique 64-bit keys (score, then lower index first), so a
// pair costs one integer compare.  Each maximum belongs to a different group of cache rows, so
// k rows score at least the k-th largest value and it is a floor for the query's top-k.
// Dependent kernels are released only at the end: a tensor-core CTA that starts early and waits
// on the same SM was measured to slow this kernel's CTAs down several times over.
__global__ void __launch_bounds__(SELECT_THREADS)
select_floor_kernel(const float* __restrict__ maxima, int n_tiles, int nq, int k, uint64_t* __restrict__ out_thr) {
  __shared__ uint64_t keys[SELECT_MAX_VALUES];
  const int q = blockIdx.x, tid = threadIdx.x;
  const int m = n_tiles * 4;
  grid_dep_wait();   // the maxima come from the previous kernel
  for (int t = tid; t < n_tiles; t += SELECT_THREADS) {
    const float4 g = *reinterpret_cast<const float4*>(maxima + ((size_t)t * nq + q) * 4);
    keys[4 * t] = make_key(g.x, (uint32_t)(4 * t));
    keys[4 * t + 1] = make_key(g.y, (uint32_t)(4 * t + 1));
    keys[4 * t + 2] = make_key(g.z, (uint32_t)(4 * t + 2));
    keys[4 * t + 3] = make_key(g.w, (uint32_t)(4 * t + 3));
  }
  if (tid == 0 && blockIdx.y == 0 && m < k) out_thr[q] = KEY_EMPTY;
  __syncthreads();
  const int i = blockIdx.y * SELECT_THREADS + tid;
  const uint64_t mine = i < m ? keys[i] : ~0ull;
  int rank = 0;   // keys larger than mine
#pragma unroll 8
  for (int j = 0; j < m; ++j) rank += keys[j] > mine ? 1 : 0;
  // admit every key whose score is >= this value: the smallest such key carries the largest slot word
  if (i < m && rank == k - 1) out_thr[q] = (mine | 0xffffffffull) - 0xffffffffull - 1;
  grid_dep_launch_dependents();
}

cudaError_t launch_select_floor(const float* maxima, int n_tiles, int nq, int k, uint64_t* out_thr, cudaStream_t st) {
  if (n_tiles < 1 || n_tiles * 4 > SELECT_MAX_VALUES || !maxima || !out_thr) return cudaErrorInvalidValue;
  const dim3 grid((unsigned)nq, (unsigned)((n_tiles * 4 + SELECT_THREADS - 1) / SELECT_THREADS));
  return launch_overlapped(select_floor_kernel, grid, dim3(SELECT_THREADS), 0, st, 1, maxima, n_tiles, nq, k, out_thr);
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
