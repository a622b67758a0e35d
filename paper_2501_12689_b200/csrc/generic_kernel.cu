// Generic CUDA-core scoring kernel: any dim (multiple of 8), up to four queries per launch.
// One warp per cache row, direct 16-byte global loads, queries read as fp32 from global
// memory.  It makes no attempt at bandwidth efficiency; it exists so that every shape has a
// correct device path and so the fast paths can be cross-checked against something simple.
#include "common.cuh"
#include "kernels.h"
#include "pipeline.cuh"

namespace icc {

constexpr int GEN_QB = 4;
constexpr int GEN_WARPS = 8;
__global__ void __launch_bounds__(GEN_WARPS * 32)
generic_score_topk_kernel(const __nv_bfloat16* __restrict__ slab, int64_t n, int dim,
                          const float* __restrict__ q_f32, int q0, int nq, int k,
                          uint64_t* __restrict__ partials, int* dev_status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint64_t* lists = reinterpret_cast<uint64_t*>(smem_raw);        // [GEN_QB][k]
  int* locks = reinterpret_cast<int*>(lists + GEN_QB * k);        // [GEN_QB]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < GEN_QB * k; i += blockDim.x) lists[i] = KEY_EMPTY;
  if (tid < GEN_QB) locks[tid] = 0;
  grid_dep_launch_dependents();
  grid_dep_wait();
  __syncthreads();

  const int nchunk = dim >> 3;
  const int qcount = min(GEN_QB, nq - q0);
  for (int64_t row = (int64_t)blockIdx.x * GEN_WARPS + warp; row < n;
       row += (int64_t)gridDim.x * GEN_WARPS) {
    float acc[GEN_QB];
#pragma unroll
    for (int qq = 0; qq < GEN_QB; ++qq) acc[qq] = 0.0f;
    const uint4* rp = reinterpret_cast<const uint4*>(slab + row * dim);
    for (int c = lane; c < nchunk; c += 32) {
      float x[8];
      bf16x8_to_f32(ld_stream_16B(rp + c), x);
#pragma unroll
      for (int qq = 0; qq < GEN_QB; ++qq) {
        if (qq < qcount) {
          const float4* qp = reinterpret_cast<const float4*>(q_f32 + (size_t)(q0 + qq) * dim) + 2 * c;
          const float4 a = __ldg(qp), b = __ldg(qp + 1);
          float s = acc[qq];
          s = fmaf(x[0], a.x, s); s = fmaf(x[1], a.y, s); s = fmaf(x[2], a.z, s); s = fmaf(x[3], a.w, s);
          s = fmaf(x[4], b.x, s); s = fmaf(x[5], b.y, s); s = fmaf(x[6], b.z, s); s = fmaf(x[7], b.w, s);
          acc[qq] = s;
        }
      }
    }
#pragma unroll
    for (int qq = 0; qq < GEN_QB; ++qq) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc[qq] += __shfl_xor_sync(FULL_MASK, acc[qq], o);
    }
#pragma unroll
    for (int qq = 0; qq < GEN_QB; ++qq) {
      if (qq < qcount) {
        const uint64_t key = make_key(acc[qq], (uint32_t)row);
        uint64_t* list = lists + qq * k;
        const uint64_t thr = *reinterpret_cast<volatile uint64_t*>(list + (k - 1));
        // lane 0 decides for the warp so that the branch is uniform by construction
        if (__shfl_sync(FULL_MASK, key > thr ? 1 : 0, 0))
          locked_insert(list, k, locks + qq, __shfl_sync(FULL_MASK, key, 0), lane, dev_status);
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < qcount * k; i += blockDim.x) {
    const int qq = i / k, j = i - qq * k;
    partials[((size_t)blockIdx.x * nq + (q0 + qq)) * k + j] = lists[i];
  }
}

cudaError_t launch_generic(const void* slab, int64_t n, int dim, const float* q_f32, int q0, int nq,
                           int k, uint64_t* partials, int n_part, int smem_bytes, int* dev_status,
                           cudaStream_t st) {
  return launch_overlapped(generic_score_topk_kernel, dim3(n_part), dim3(GEN_WARPS * 32), (size_t)smem_bytes, st, 1,
                           static_cast<const __nv_bfloat16*>(slab), n, dim, q_f32, q0, nq, k, partials, dev_status);
}

}  // namespace icc
