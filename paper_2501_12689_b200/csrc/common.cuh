// Device helpers shared by the scoring and merge kernels: the packed (score, slot) key and
// the warp-cooperative sorted insert that every partial top-k list uses.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace icc {

constexpr unsigned FULL_MASK = 0xffffffffu;
constexpr uint64_t KEY_EMPTY = 0ull;  // smaller than every real key

// Status word values written by kernels whose bounded waits expire (device -> host).
enum : int { DEV_OK = 0, DEV_TIMEOUT_LOCK = 1, DEV_TIMEOUT_MBAR = 2, DEV_CHECK_FAILED = 3 };

// Monotone map from fp32 scores to unsigned integers (-0 is folded onto +0 first so that
// equal scores give equal keys).
__device__ __forceinline__ uint32_t score_to_ord(float s) {
  s += 0.0f;
  uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ord_to_score(uint32_t o) {
  uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
  return __uint_as_float(u);
}
// One 64-bit key per candidate: larger key = better candidate (higher score; on equal score
// the earlier slot).  A single integer compare therefore orders candidates everywhere.
__device__ __forceinline__ uint64_t make_key(float score, uint32_t slot) {
  return ((uint64_t)score_to_ord(score) << 32) | (uint64_t)(0xffffffffu - slot);
}
__device__ __forceinline__ uint32_t key_slot(uint64_t key) { return 0xffffffffu - (uint32_t)key; }
__device__ __forceinline__ float key_score(uint64_t key) { return ord_to_score((uint32_t)(key >> 32)); }

constexpr int MAX_K = 128;  // must equal IC_MAX_K

// Record that a bounded wait expired.  The status word lives in mapped pinned host memory,
// so a plain store followed by a system-scope fence is what the host polls.
__device__ __forceinline__ void report_status(int* dev_status, int code) {
  *reinterpret_cast<volatile int*>(dev_status) = code;
  __threadfence_system();
}

// Index checks of the debug build (-DIC_CACHE_DEBUG_CHECKS, libic_cache_debug.so): a failed check
// writes DEV_CHECK_FAILED to the status word, which the host reports like an expired wait; it never
// traps.  In the normal build the macro is empty.
#ifdef IC_CACHE_DEBUG_CHECKS
#define ICC_CHECK(cond, dev_status)                                        \
  do {                                                                     \
    if (!(cond)) icc::report_status((dev_status), icc::DEV_CHECK_FAILED);  \
  } while (0)
#else
#define ICC_CHECK(cond, dev_status) \
  do {                              \
  } while (0)
#endif

// Insert `key` into a descending list of k entries in shared memory, dropping the last one.
// All 32 lanes of the warp call this with the same arguments; the caller guarantees that no
// other warp touches the list meanwhile.  A key not larger than the last entry changes
// nothing.  Returns the new last entry (the list's admission threshold).
__device__ __forceinline__ uint64_t warp_sorted_insert(uint64_t* list, int k, uint64_t key, int lane) {
  uint64_t nv[MAX_K / 32];
#pragma unroll
  for (int t = 0; t < MAX_K / 32; ++t) {
    const int i = t * 32 + lane;
    nv[t] = 0;
    if (i < k) {
      const uint64_t cur = list[i];
      const uint64_t prev = (i > 0) ? list[i - 1] : ~0ull;
      nv[t] = (cur > key) ? cur : ((prev > key) ? key : prev);
    }
  }
  __syncwarp();
#pragma unroll
  for (int t = 0; t < MAX_K / 32; ++t) {
    const int i = t * 32 + lane;
    if (i < k) list[i] = nv[t];
  }
  __syncwarp();
  return list[k - 1];
}

constexpr int LOCK_SPIN_LIMIT = 1 << 22;

// warp_sorted_insert under a per-list spin lock, for lists shared by the warps of a CTA.
// The wait is bounded: if the lock cannot be taken the candidate is dropped and the status
// word records it.  All 32 lanes call this with the same arguments.
__device__ __forceinline__ void locked_insert(uint64_t* list, int k, int* lock, uint64_t key,
                                              int lane, int* dev_status) {
  int ok = 1;
  if (lane == 0) {
    int spins = 0;
    while (atomicCAS(lock, 0, 1) != 0) {
      if (++spins > LOCK_SPIN_LIMIT) {
        ok = 0;
        break;
      }
      __nanosleep(32);
    }
  }
  ok = __shfl_sync(FULL_MASK, ok, 0);
  if (!ok) {
    if (lane == 0) report_status(dev_status, DEV_TIMEOUT_LOCK);
    return;
  }
  __threadfence_block();
  warp_sorted_insert(list, k, key, lane);
  __threadfence_block();
  if (lane == 0) atomicExch(lock, 0);
}

// Tournament over the heads of sorted lists (list p starts at cand[p * stride], k entries each),
// run by one warp; the winners go to win_key in order.  Lane l owns lists l, l+32,
// ...; the current head of each owned list is kept in a register, so a round costs a few
// compares, two warp max-reductions (score word, then slot word) and, for the winning lane
// only, one shared-memory load of its list's next entry.  Returns the number of winners.
template <int LPL>
__device__ __forceinline__ int tournament_in_registers(const uint64_t* cand, int stride, int n_part, int k,
                                                       int lane, uint64_t* win_key) {
  uint64_t head[LPL];
  int idx[LPL];
#pragma unroll
  for (int t = 0; t < LPL; ++t) {
    const int p = lane + 32 * t;
    head[t] = (p < n_part) ? cand[(size_t)p * stride] : KEY_EMPTY;
    idx[t] = 0;
  }
  int r = 0;
  for (; r < k; ++r) {
    uint64_t best = head[0];
#pragma unroll
    for (int t = 1; t < LPL; ++t) best = head[t] > best ? head[t] : best;
    const uint32_t hi = (uint32_t)(best >> 32);
    const uint32_t top_hi = __reduce_max_sync(FULL_MASK, hi);
    if (top_hi == 0) break;  // every list exhausted (warp-uniform)
    const uint32_t lo = (hi == top_hi) ? (uint32_t)best : 0u;
    const uint32_t top_lo = __reduce_max_sync(FULL_MASK, lo);
    if (hi == top_hi && lo == top_lo) {  // keys are unique, so exactly one lane wins
      win_key[r] = best;
#pragma unroll
      for (int t = 0; t < LPL; ++t) {
        if (head[t] == best) {
          idx[t] += 1;
          head[t] = (idx[t] < k) ? cand[(size_t)(lane + 32 * t) * stride + idx[t]] : KEY_EMPTY;
        }
      }
    }
  }
  return r;
}

// Unpack eight bf16 values held in a 16-byte vector into fp32.
__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float* x) {
  x[0] = __uint_as_float(v.x << 16);
  x[1] = __uint_as_float(v.x & 0xffff0000u);
  x[2] = __uint_as_float(v.y << 16);
  x[3] = __uint_as_float(v.y & 0xffff0000u);
  x[4] = __uint_as_float(v.z << 16);
  x[5] = __uint_as_float(v.z & 0xffff0000u);
  x[6] = __uint_as_float(v.w << 16);
  x[7] = __uint_as_float(v.w & 0xffff0000u);
}

// Streaming 16-byte global load that does not allocate in L1.
__device__ __forceinline__ uint4 ld_stream_16B(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

}  // namespace icc
