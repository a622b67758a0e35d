// Row conversion used by insert (into the slab) and by query preparation (into the query
// staging buffers): optional fp32 L2 normalisation, then round-to-nearest-even to bf16.
#include "common.cuh"
#include "kernels.h"
#include "pipeline.cuh"

namespace icc {

constexpr int CONV_WARPS = 8;
constexpr int CONV_MAX_CHUNKS = 16;  // 16 chunks * 32 lanes * 8 elements = 4096 = IC_MAX_DIM

// One warp per row.  Lane l owns the 8-element chunks l, l+32, ... of the row.
template <bool IN_F32>
__global__ void __launch_bounds__(CONV_WARPS * 32)
convert_rows_kernel(const void* __restrict__ in, int64_t nrows, int dim, int normalize,
                    __nv_bfloat16* __restrict__ out_bf16, float* __restrict__ out_f32,
                    int64_t pad_rows, const int64_t* __restrict__ ids_in, int64_t* __restrict__ ids_out) {
  grid_dep_launch_dependents();
  grid_dep_wait();   // the destination may still be read by the previous kernel in the stream
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * CONV_WARPS + (threadIdx.x >> 5);
  if (row >= pad_rows) return;
  const int nchunk = dim >> 3;
  uint4* orow = reinterpret_cast<uint4*>(out_bf16 + row * dim);
  if (row >= nrows) {  // zero padding rows
    for (int c = lane; c < nchunk; c += 32) orow[c] = make_uint4(0, 0, 0, 0);
    return;
  }
  if (ids_in && lane == 0) ids_out[row] = ids_in[row];
  float x[CONV_MAX_CHUNKS / 1][8];
  float ss = 0.0f;
#pragma unroll
  for (int t = 0; t < CONV_MAX_CHUNKS; ++t) {
    const int c = t * 32 + lane;
    if (c < nchunk) {
      if (IN_F32) {
        const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(in) + row * dim) + 2 * c;
        const float4 a = p[0], b = p[1];
        x[t][0] = a.x; x[t][1] = a.y; x[t][2] = a.z; x[t][3] = a.w;
        x[t][4] = b.x; x[t][5] = b.y; x[t][6] = b.z; x[t][7] = b.w;
      } else {
        const uint4 v = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(in) + row * dim)[c];
        bf16x8_to_f32(v, x[t]);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) ss = fmaf(x[t][e], x[t][e], ss);
    }
  }
  float scale = 1.0f;
  if (normalize) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(FULL_MASK, ss, o);
    scale = (ss > 0.0f) ? (1.0f / sqrtf(ss)) : 0.0f;
  }
#pragma unroll
  for (int t = 0; t < CONV_MAX_CHUNKS; ++t) {
    const int c = t * 32 + lane;
    if (c < nchunk) {
      uint32_t w[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const __nv_bfloat16 lo = __float2bfloat16_rn(x[t][2 * e] * scale);
        const __nv_bfloat16 hi = __float2bfloat16_rn(x[t][2 * e + 1] * scale);
        w[e] = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
      }
      const uint4 v = make_uint4(w[0], w[1], w[2], w[3]);
      orow[c] = v;
      if (out_f32) {
        float y[8];
        bf16x8_to_f32(v, y);
        float4* q = reinterpret_cast<float4*>(out_f32 + row * dim) + 2 * c;
        q[0] = make_float4(y[0], y[1], y[2], y[3]);
        q[1] = make_float4(y[4], y[5], y[6], y[7]);
      }
    }
  }
}

cudaError_t launch_convert_rows(const void* in, int in_is_f32, int64_t nrows, int dim, int normalize,
                                void* out_bf16, float* out_f32, int64_t pad_rows, const int64_t* ids_in,
                                int64_t* ids_out, cudaStream_t st) {
  if (pad_rows < nrows) pad_rows = nrows;
  if (pad_rows == 0) return cudaSuccess;
  const unsigned blocks = (unsigned)((pad_rows + CONV_WARPS - 1) / CONV_WARPS);
  if (in_is_f32)
    return launch_overlapped(convert_rows_kernel<true>, dim3(blocks), dim3(CONV_WARPS * 32), 0, st, 1, in, nrows, dim,
                             normalize, static_cast<__nv_bfloat16*>(out_bf16), out_f32, pad_rows, ids_in, ids_out);
  return launch_overlapped(convert_rows_kernel<false>, dim3(blocks), dim3(CONV_WARPS * 32), 0, st, 1, in, nrows, dim,
                           normalize, static_cast<__nv_bfloat16*>(out_bf16), out_f32, pad_rows, ids_in, ids_out);
}

// Eviction support.  find_ids_kernel lists the slots whose id is one of `wanted` (sorted
// ascending, n_wanted entries): one thread per cache row, binary search, matches appended
// through an atomic counter (their order is arbitrary; the host sorts them).
__global__ void __launch_bounds__(256)
find_ids_kernel(const int64_t* __restrict__ ids, int64_t n, const int64_t* __restrict__ wanted, int64_t n_wanted,
                int64_t* __restrict__ match_slots, unsigned long long* __restrict__ match_count, int64_t cap) {
  grid_dep_launch_dependents();
  grid_dep_wait();
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int64_t id = ids[i];
  int64_t lo = 0, hi = n_wanted;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (wanted[mid] < id) lo = mid + 1;
    else hi = mid;
  }
  if (lo < n_wanted && wanted[lo] == id) {
    const unsigned long long pos = atomicAdd(match_count, 1ull);
    if ((int64_t)pos < cap) match_slots[pos] = i;
  }
}

// Copy whole rows (and their ids) inside the slab: row src[i] -> row dst[i].  The two sets are
// disjoint (tail rows move into vacated slots), so rows can move in parallel.
__global__ void __launch_bounds__(CONV_WARPS * 32)
move_rows_kernel(__nv_bfloat16* __restrict__ slab, int64_t* __restrict__ ids, float* __restrict__ utility,
                 const int64_t* __restrict__ src, const int64_t* __restrict__ dst, int64_t nmoves, int dim) {
  grid_dep_launch_dependents();
  grid_dep_wait();
  const int lane = threadIdx.x & 31;
  const int64_t i = (int64_t)blockIdx.x * CONV_WARPS + (threadIdx.x >> 5);
  if (i >= nmoves) return;
  const int64_t s = src[i], d = dst[i];
  const uint4* from = reinterpret_cast<const uint4*>(slab + s * dim);
  uint4* to = reinterpret_cast<uint4*>(slab + d * dim);
  for (int c = lane; c < (dim >> 3); c += 32) to[c] = from[c];
  if (lane == 0) {
    ids[d] = ids[s];
    if (utility) utility[d] = utility[s];
  }
}

cudaError_t launch_find_ids(const int64_t* ids, int64_t n, const int64_t* wanted, int64_t n_wanted, int64_t* match_slots,
                            unsigned long long* match_count, int64_t cap, cudaStream_t st) {
  if (n == 0 || n_wanted == 0) return cudaSuccess;
  const unsigned blocks = (unsigned)((n + 255) / 256);
  return launch_overlapped(find_ids_kernel, dim3(blocks), dim3(256), 0, st, 1, ids, n, wanted, n_wanted, match_slots,
                           match_count, cap);
}

cudaError_t launch_move_rows(void* slab, int64_t* ids, float* utility, const int64_t* src, const int64_t* dst,
                             int64_t nmoves, int dim, cudaStream_t st) {
  if (nmoves == 0) return cudaSuccess;
  const unsigned blocks = (unsigned)((nmoves + CONV_WARPS - 1) / CONV_WARPS);
  return launch_overlapped(move_rows_kernel, dim3(blocks), dim3(CONV_WARPS * 32), 0, st, 1,
                           static_cast<__nv_bfloat16*>(slab), ids, utility, src, dst, nmoves, dim);
}

// Per-entry utility (paper Sec. 4.3, "Example Manager": the efficiency gain of an example, kept as
// a moving average that is decayed over time).  utility_add_kernel: one thread per cache row looks
// its id up in `wanted` (sorted ascending, equal ids kept in the caller's order) and adds the gains
// of all matching entries, one fp32 addition each, in that order.  utility_scale_kernel multiplies
// every entry's utility by one factor.
__global__ void __launch_bounds__(256)
utility_add_kernel(const int64_t* __restrict__ ids, int64_t n, const int64_t* __restrict__ wanted,
                   const float* __restrict__ gains, int64_t n_wanted, float* __restrict__ utility) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int64_t id = ids[i];
  int64_t lo = 0, hi = n_wanted;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (wanted[mid] < id) lo = mid + 1;
    else hi = mid;
  }
  if (lo < n_wanted && wanted[lo] == id) {
    float u = utility[i];
    for (; lo < n_wanted && wanted[lo] == id; ++lo) u += gains[lo];
    utility[i] = u;
  }
}

__global__ void __launch_bounds__(256) utility_scale_kernel(float* __restrict__ utility, int64_t n, float factor) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) utility[i] *= factor;
}

cudaError_t launch_utility_add(const int64_t* ids, int64_t n, const int64_t* wanted, const float* gains, int64_t n_wanted,
                               float* utility, cudaStream_t st) {
  if (n == 0 || n_wanted == 0) return cudaSuccess;
  utility_add_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(ids, n, wanted, gains, n_wanted, utility);
  return cudaGetLastError();
}

cudaError_t launch_utility_scale(float* utility, int64_t n, float factor, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  utility_scale_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(utility, n, factor);
  return cudaGetLastError();
}

// Exercise of the bounded-wait path: one thread waits, with a short limit, on an mbarrier that
// nothing ever completes, then reports the expiry exactly as the scoring kernels would.
__global__ void wait_limit_probe_kernel(long long limit_cycles, int* dev_status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    mbar_fence_init();
    if (!mbar_wait(&bar, 0, &abort_flag, limit_cycles)) report_status(dev_status, DEV_TIMEOUT_MBAR);
  }
}

cudaError_t launch_wait_limit_probe(long long limit_cycles, int* dev_status, cudaStream_t st) {
  wait_limit_probe_kernel<<<1, 32, 0, st>>>(limit_cycles, dev_status);
  return cudaGetLastError();
}

}  // namespace icc
