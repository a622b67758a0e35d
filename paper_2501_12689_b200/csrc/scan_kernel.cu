// Scan path: HBM-bound CUDA-core scoring for small query batches (1, 2 or 4 queries per pass).
//
// One persistent CTA per SM.  A producer warp streams contiguous 32-row pieces of the slab
// into a shared-memory ring with bulk async copies (one copy per piece, completion counted on
// an mbarrier); eight consumer warps each take four rows of a piece, read them back with
// conflict-free 16-byte shared loads (lane l owns elements [8l, 8l+8) of every 256-element
// span), multiply against queries held in registers as fp32, and reduce across the warp with
// a transposing butterfly (one shuffle per (row, query) instead of five).  Candidates that
// beat the warp's current k-th best go into the warp's own sorted list for that query (no
// locks); when the scan ends, one warp per query merges the eight lists into the CTA's list.
#include "common.cuh"
#include "kernels.h"
#include "pipeline.cuh"

namespace icc {

constexpr int SCAN_CONSUMER_WARPS = 8;
constexpr int SCAN_THREADS = (SCAN_CONSUMER_WARPS + 1) * 32;
constexpr int SCAN_ROWS_PER_WARP = 4;
constexpr int SCAN_STAGE_ROWS = SCAN_CONSUMER_WARPS * SCAN_ROWS_PER_WARP;  // 32
constexpr int SCAN_MAX_STAGES = 8;
constexpr int SCAN_LISTS_OFFSET = 2048;
constexpr int SCAN_MAX_QB = 4;

struct ScanSmemHeader {
  uint64_t full[SCAN_MAX_STAGES];
  uint64_t empty[SCAN_MAX_STAGES];
  int abort_flag;
};

// Cross-lane sum of V per-lane values so that afterwards lane l holds, in v[0], the total of
// value number (l >> (5 - log2 V)).  V - 1 + (5 - log2 V) shuffles instead of 5 V.
template <int V>
__device__ __forceinline__ float transpose_reduce(float (&v)[V], int lane) {
  int o = 16;
#pragma unroll
  for (int half = V / 2; half >= 1; half /= 2, o /= 2) {
    const bool upper = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < half; ++i) {
      const float send = upper ? v[i] : v[i + half];
      const float keep = upper ? v[i + half] : v[i];
      v[i] = keep + __shfl_xor_sync(FULL_MASK, send, o);
    }
  }
  for (; o >= 1; o /= 2) v[0] += __shfl_xor_sync(FULL_MASK, v[0], o);
  return v[0];
}

template <int QB, int NCHUNK>
__global__ void __launch_bounds__(SCAN_THREADS, 1)
scan_score_topk_kernel(const __nv_bfloat16* __restrict__ slab, int64_t n, int dim,
                       const float* __restrict__ q_f32, int q0, int nq, int k,
                       uint64_t* __restrict__ partials, int n_stages, int* dev_status) {
  extern __shared__ __align__(128) unsigned char smem[];
  ScanSmemHeader* hdr = reinterpret_cast<ScanSmemHeader*>(smem);
  uint64_t* lists = reinterpret_cast<uint64_t*>(smem + SCAN_LISTS_OFFSET);        // [8 warps][SCAN_MAX_QB][k]
  unsigned char* ring = smem + SCAN_LISTS_OFFSET + SCAN_CONSUMER_WARPS * SCAN_MAX_QB * k * 8;
  const int stage_bytes = SCAN_STAGE_ROWS * dim * 2;
  const int row_bytes = dim * 2;
  volatile int* abort_flag = &hdr->abort_flag;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&hdr->full[s], 1);
      mbar_init(&hdr->empty[s], SCAN_CONSUMER_WARPS);
    }
    hdr->abort_flag = 0;
    mbar_fence_init();
  }
  for (int i = tid; i < SCAN_CONSUMER_WARPS * SCAN_MAX_QB * k; i += SCAN_THREADS) lists[i] = KEY_EMPTY;
  grid_dep_launch_dependents();
  grid_dep_wait();   // queries and newly inserted rows come from earlier kernels in the stream
  __syncthreads();

  const int64_t n_pieces = (n + SCAN_STAGE_ROWS - 1) / SCAN_STAGE_ROWS;
  const int qcount = min(QB, nq - q0);

  if (warp == SCAN_CONSUMER_WARPS) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      int64_t it = 0;
      bool ok = true;
      for (int64_t piece = blockIdx.x; piece < n_pieces && ok; piece += gridDim.x, ++it) {
        const int s = (int)(it % n_stages);
        const uint32_t ph = (uint32_t)((it / n_stages) & 1);
        ok = mbar_wait(&hdr->empty[s], ph ^ 1u, abort_flag);
        if (!ok) break;
        const int64_t row0 = piece * SCAN_STAGE_ROWS;
        const uint32_t bytes = (uint32_t)(min((int64_t)SCAN_STAGE_ROWS, n - row0) * row_bytes);
        mbar_arrive_expect_tx(&hdr->full[s], bytes);
        bulk_load(ring + (size_t)s * stage_bytes, slab + row0 * dim, bytes, &hdr->full[s]);
      }
      if (!ok) {
        report_status(dev_status, DEV_TIMEOUT_MBAR);
        // copies already issued still land in this CTA's shared memory: wait for them
        // (bounded) before the CTA may exit
        for (int64_t j = (it > n_stages ? it - n_stages : 0); j < it; ++j) {
          const int s = (int)(j % n_stages);
          const long long t0 = clock64();
          while (!mbar_try_wait(&hdr->full[s], (uint32_t)((j / n_stages) & 1)) &&
                 clock64() - t0 < WAIT_LIMIT_CYCLES) {
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ consumers
    // queries in registers: lane l holds components [256 t + 8 l, 256 t + 8 l + 8) of each query
    float qreg[QB][NCHUNK][8];
#pragma unroll
    for (int qq = 0; qq < QB; ++qq) {
#pragma unroll
      for (int t = 0; t < NCHUNK; ++t) {
        const int c = t * 32 + lane;
        const bool live = (qq < qcount) && (c * 8 < dim);
        const float4* qp = reinterpret_cast<const float4*>(q_f32 + (size_t)(q0 + (live ? qq : 0)) * dim) + 2 * (live ? c : 0);
        const float4 a = live ? __ldg(qp) : make_float4(0, 0, 0, 0);
        const float4 b = live ? __ldg(qp + 1) : make_float4(0, 0, 0, 0);
        qreg[qq][t][0] = a.x; qreg[qq][t][1] = a.y; qreg[qq][t][2] = a.z; qreg[qq][t][3] = a.w;
        qreg[qq][t][4] = b.x; qreg[qq][t][5] = b.y; qreg[qq][t][6] = b.z; qreg[qq][t][7] = b.w;
      }
    }
    constexpr int V = SCAN_ROWS_PER_WARP * QB;     // values reduced together
    constexpr int SHIFT = (V == 16) ? 1 : (V == 8) ? 2 : 3;   // lane -> value number
    const int my_val = lane >> SHIFT;
    const int my_row = my_val / QB;                // row within the warp's four
    const int my_q = my_val % QB;                  // query this lane reports for
    const bool reporter = (lane & ((1 << SHIFT) - 1)) == 0 && my_q < qcount;
    uint64_t* warp_lists = lists + (size_t)warp * SCAN_MAX_QB * k;   // this warp's [SCAN_MAX_QB][k]
    uint64_t thr = KEY_EMPTY;                                       // k-th best of list my_q

    int64_t it = 0;
    bool ok = true;
    for (int64_t piece = blockIdx.x; piece < n_pieces; piece += gridDim.x, ++it) {
      const int s = (int)(it % n_stages);
      const uint32_t ph = (uint32_t)((it / n_stages) & 1);
      ok = mbar_wait(&hdr->full[s], ph, abort_flag);
      if (!ok) break;
      const unsigned char* base = ring + (size_t)s * stage_bytes + (size_t)(warp * SCAN_ROWS_PER_WARP) * row_bytes;
      float acc[V];
#pragma unroll
      for (int i = 0; i < V; ++i) acc[i] = 0.0f;
#pragma unroll
      for (int t = 0; t < NCHUNK; ++t) {
        const int c = t * 32 + lane;
        const bool live = c * 8 < dim;
#pragma unroll
        for (int r = 0; r < SCAN_ROWS_PER_WARP; ++r) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (live) v = *reinterpret_cast<const uint4*>(base + (size_t)r * row_bytes + (size_t)c * 16);
          float x[8];
          bf16x8_to_f32(v, x);
#pragma unroll
          for (int qq = 0; qq < QB; ++qq) {
            float a = acc[r * QB + qq];
#pragma unroll
            for (int e = 0; e < 8; ++e) a = fmaf(x[e], qreg[qq][t][e], a);
            acc[r * QB + qq] = a;
          }
        }
      }
      // all of this warp's reads of the stage are done: hand the slot back early
      __syncwarp();
      if (lane == 0) mbar_arrive(&hdr->empty[s]);

      const float score = transpose_reduce<V>(acc, lane);
      const int64_t row = piece * SCAN_STAGE_ROWS + warp * SCAN_ROWS_PER_WARP + my_row;
      const uint64_t key = make_key(score, (uint32_t)row);
      ICC_CHECK(my_q < QB && piece < n_pieces, dev_status);
      const bool hit = reporter && row < n && key > thr;
      unsigned hits = __ballot_sync(FULL_MASK, hit);
      while (hits) {
        const int src = __ffs(hits) - 1;
        hits &= hits - 1;
        const uint64_t hkey = __shfl_sync(FULL_MASK, key, src);
        const int hq = __shfl_sync(FULL_MASK, my_q, src);
        const uint64_t new_thr = warp_sorted_insert(warp_lists + hq * k, k, hkey, lane);
        if (my_q == hq) thr = new_thr;
      }
    }
    if (!ok && lane == 0) report_status(dev_status, DEV_TIMEOUT_MBAR);
  }
  __syncthreads();
  // warp qq merges the eight warps' lists of query qq and writes the CTA's partial list
  if (warp < qcount) {
    uint64_t* dst = partials + ((size_t)blockIdx.x * nq + (q0 + warp)) * k;
    const int won = tournament_in_registers<1>(lists + (size_t)warp * k, SCAN_MAX_QB * k, SCAN_CONSUMER_WARPS, k, lane, dst);
    for (int i = won + lane; i < k; i += 32) dst[i] = KEY_EMPTY;
  }
}

// Two-level search: the same bulk-copy pipeline over one piece of one probed cluster.  CTA b scores
// query b / (n_probe * n_split) against piece (b % n_split) of its (b / n_split % n_probe)-th probed
// cluster, whose members are one contiguous run of `sorted_rows` (row p = cache row order[p]).  A
// row's slot is looked up in the member list only when its score can enter a list.  Output: one
// sorted partial list per CTA at partials[(j * n_split + s) * nq + q].
template <int NCHUNK>
__global__ void __launch_bounds__(SCAN_THREADS, 1)
cluster_stream_topk_kernel(const __nv_bfloat16* __restrict__ sorted_rows, int dim, const float* __restrict__ q_f32, int nq,
                           int k, const int64_t* __restrict__ probes, int n_probe, int n_split,
                           const int* __restrict__ offsets, const int* __restrict__ order,
                           uint64_t* __restrict__ partials, int n_stages, int* dev_status) {
  extern __shared__ __align__(128) unsigned char smem[];
  ScanSmemHeader* hdr = reinterpret_cast<ScanSmemHeader*>(smem);
  uint64_t* lists = reinterpret_cast<uint64_t*>(smem + SCAN_LISTS_OFFSET);        // [8 warps][k]
  unsigned char* ring = smem + SCAN_LISTS_OFFSET + ((SCAN_CONSUMER_WARPS * k * 8 + 127) & ~127);
  const int stage_bytes = SCAN_STAGE_ROWS * dim * 2;
  const int row_bytes = dim * 2;
  volatile int* abort_flag = &hdr->abort_flag;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_query = n_probe * n_split;
  const int q = blockIdx.x / per_query, l = blockIdx.x - q * per_query;
  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&hdr->full[s], 1);
      mbar_init(&hdr->empty[s], SCAN_CONSUMER_WARPS);
    }
    hdr->abort_flag = 0;
    mbar_fence_init();
  }
  for (int i = tid; i < SCAN_CONSUMER_WARPS * k; i += SCAN_THREADS) lists[i] = KEY_EMPTY;
  grid_dep_launch_dependents();
  grid_dep_wait();   // probes and the prepared query come from earlier kernels in the stream
  __syncthreads();

  // member-list positions [m0, m1) of this piece (none when the probe is padding)
  int64_t m0 = 0, m1 = 0;
  {
    const int64_t c = probes[(size_t)q * n_probe + l / n_split];
    if (c >= 0) {
      const int sp = l % n_split;
      const int64_t o0 = offsets[c], len = offsets[c + 1] - o0;
      m0 = o0 + len * sp / n_split;
      m1 = o0 + len * (sp + 1) / n_split;
    }
  }
  const int64_t n_rows = m1 - m0;
  const int64_t n_pieces = (n_rows + SCAN_STAGE_ROWS - 1) / SCAN_STAGE_ROWS;

  if (warp == SCAN_CONSUMER_WARPS) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      int64_t it = 0;
      bool ok = true;
      for (int64_t piece = 0; piece < n_pieces && ok; ++piece, ++it) {
        const int s = (int)(it % n_stages);
        const uint32_t ph = (uint32_t)((it / n_stages) & 1);
        ok = mbar_wait(&hdr->empty[s], ph ^ 1u, abort_flag);
        if (!ok) break;
        const int64_t row0 = piece * SCAN_STAGE_ROWS;
        const uint32_t bytes = (uint32_t)(min((int64_t)SCAN_STAGE_ROWS, n_rows - row0) * row_bytes);
        mbar_arrive_expect_tx(&hdr->full[s], bytes);
        bulk_load(ring + (size_t)s * stage_bytes, sorted_rows + (m0 + row0) * dim, bytes, &hdr->full[s]);
      }
      if (!ok) {
        report_status(dev_status, DEV_TIMEOUT_MBAR);
        // copies already issued still land in this CTA's shared memory: wait for them (bounded)
        for (int64_t j = (it > n_stages ? it - n_stages : 0); j < it; ++j) {
          const int s = (int)(j % n_stages);
          const long long t0 = clock64();
          while (!mbar_try_wait(&hdr->full[s], (uint32_t)((j / n_stages) & 1)) &&
                 clock64() - t0 < WAIT_LIMIT_CYCLES) {
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ consumers
    float qreg[NCHUNK][8];
#pragma unroll
    for (int t = 0; t < NCHUNK; ++t) {
      const int c = t * 32 + lane;
      const bool live = c * 8 < dim;
      const float4* qp = reinterpret_cast<const float4*>(q_f32 + (size_t)q * dim) + 2 * (live ? c : 0);
      const float4 a = live ? __ldg(qp) : make_float4(0, 0, 0, 0);
      const float4 b = live ? __ldg(qp + 1) : make_float4(0, 0, 0, 0);
      qreg[t][0] = a.x; qreg[t][1] = a.y; qreg[t][2] = a.z; qreg[t][3] = a.w;
      qreg[t][4] = b.x; qreg[t][5] = b.y; qreg[t][6] = b.z; qreg[t][7] = b.w;
    }
    constexpr int V = SCAN_ROWS_PER_WARP;          // four values reduced together: lane -> row lane >> 3
    const int my_row = lane >> 3;
    const bool reporter = (lane & 7) == 0;
    uint64_t* my_list = lists + (size_t)warp * k;
    uint64_t thr = KEY_EMPTY;
    bool ok = true;
    for (int64_t piece = 0; piece < n_pieces; ++piece) {
      const int s = (int)(piece % n_stages);
      const uint32_t ph = (uint32_t)((piece / n_stages) & 1);
      ok = mbar_wait(&hdr->full[s], ph, abort_flag);
      if (!ok) break;
      const unsigned char* base = ring + (size_t)s * stage_bytes + (size_t)(warp * SCAN_ROWS_PER_WARP) * row_bytes;
      float acc[V];
#pragma unroll
      for (int i = 0; i < V; ++i) acc[i] = 0.0f;
#pragma unroll
      for (int t = 0; t < NCHUNK; ++t) {
        const int c = t * 32 + lane;
        const bool live = c * 8 < dim;
#pragma unroll
        for (int r = 0; r < SCAN_ROWS_PER_WARP; ++r) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (live) v = *reinterpret_cast<const uint4*>(base + (size_t)r * row_bytes + (size_t)c * 16);
          float x[8];
          bf16x8_to_f32(v, x);
          float a = acc[r];
#pragma unroll
          for (int e = 0; e < 8; ++e) a = fmaf(x[e], qreg[t][e], a);
          acc[r] = a;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&hdr->empty[s]);

      const float score = transpose_reduce<V>(acc, lane);
      const int64_t pos = m0 + piece * SCAN_STAGE_ROWS + warp * SCAN_ROWS_PER_WARP + my_row;
      // rows past the piece hold whatever the stage held before; a score (NaN included) below the
      // list's last score cannot enter
      const bool maybe = reporter && pos < m1 && score_to_ord(score) >= (uint32_t)(thr >> 32) && score == score;
      uint64_t key = KEY_EMPTY;
      ICC_CHECK(!maybe || (pos >= m0 && pos < m1), dev_status);
      if (maybe) key = make_key(score, (uint32_t)order[pos]);
      unsigned hits = __ballot_sync(FULL_MASK, maybe && key > thr);
      while (hits) {
        const int src = __ffs(hits) - 1;
        hits &= hits - 1;
        const uint64_t hkey = __shfl_sync(FULL_MASK, key, src);
        thr = warp_sorted_insert(my_list, k, hkey, lane);
      }
    }
    if (!ok && lane == 0) report_status(dev_status, DEV_TIMEOUT_MBAR);
  }
  __syncthreads();
  if (warp == 0) {
    uint64_t* dst = partials + ((size_t)l * nq + q) * k;
    const int won = tournament_in_registers<1>(lists, k, SCAN_CONSUMER_WARPS, k, lane, dst);
    for (int i = won + lane; i < k; i += 32) dst[i] = KEY_EMPTY;
  }
}

template <int NCHUNK>
static cudaError_t launch_cluster_stream_t(const ClusterStreamParams& p, cudaStream_t st) {
  return launch_overlapped(cluster_stream_topk_kernel<NCHUNK>, dim3((unsigned)(p.nq * p.n_probe * p.n_split)), dim3(SCAN_THREADS),
                           (size_t)p.smem_bytes, st, 1, static_cast<const __nv_bfloat16*>(p.sorted_rows), p.dim, p.q_f32, p.nq,
                           p.k, p.probes, p.n_probe, p.n_split, p.offsets, p.order, p.partials, p.n_stages, p.dev_status);
}

int cluster_stream_smem_bytes(int dim, int k, int n_stages) {
  return SCAN_LISTS_OFFSET + ((SCAN_CONSUMER_WARPS * k * 8 + 127) & ~127) + n_stages * SCAN_STAGE_ROWS * dim * 2;
}

cudaError_t launch_cluster_stream(const ClusterStreamParams& p, cudaStream_t st) {
  if (p.n_stages < 2 || p.n_stages > SCAN_MAX_STAGES || p.dim > 1024 || p.nq < 1 || p.n_probe < 1 || p.n_split < 1)
    return cudaErrorInvalidValue;
  if (cluster_stream_smem_bytes(p.dim, p.k, p.n_stages) > p.smem_bytes) return cudaErrorInvalidValue;
  switch ((p.dim + 255) / 256) {
    case 1: return launch_cluster_stream_t<1>(p, st);
    case 2: return launch_cluster_stream_t<2>(p, st);
    case 3: return launch_cluster_stream_t<3>(p, st);
    case 4: return launch_cluster_stream_t<4>(p, st);
    default: return cudaErrorInvalidValue;
  }
}

template <int QB, int NCHUNK>
static cudaError_t launch_scan_t(const ScanParams& p, cudaStream_t st) {
  return launch_overlapped(scan_score_topk_kernel<QB, NCHUNK>, dim3(p.n_part), dim3(SCAN_THREADS), (size_t)p.smem_bytes,
                           st, 1, static_cast<const __nv_bfloat16*>(p.slab), p.n, p.dim, p.q_f32, p.q0, p.nq, p.k,
                           p.partials, p.n_stages, p.dev_status);
}

template <int QB>
static cudaError_t launch_scan_q(const ScanParams& p, cudaStream_t st) {
  const int nchunk = (p.dim + 255) / 256;
  switch (nchunk) {
    case 1: return launch_scan_t<QB, 1>(p, st);
    case 2: return launch_scan_t<QB, 2>(p, st);
    case 3: return launch_scan_t<QB, 3>(p, st);
    case 4: return launch_scan_t<QB, 4>(p, st);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_scan(const ScanParams& p, cudaStream_t st) {
  if (p.rows_per_stage != SCAN_STAGE_ROWS || p.n_stages < 2 || p.n_stages > SCAN_MAX_STAGES) return cudaErrorInvalidValue;
  if (sizeof(ScanSmemHeader) > SCAN_LISTS_OFFSET) return cudaErrorInvalidValue;
  switch (p.qb) {
    case 1: return launch_scan_q<1>(p, st);
    case 2: return launch_scan_q<2>(p, st);
    case 4: return launch_scan_q<4>(p, st);
    default: return cudaErrorInvalidValue;
  }
}

template <int QB, int NCHUNK>
static cudaError_t scan_set_attr(int bytes) {
  return cudaFuncSetAttribute(scan_score_topk_kernel<QB, NCHUNK>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}

cudaError_t scan_configure(int smem_optin) {
  cudaError_t e = cudaSuccess;
#define ICC_SET(QB, NC)                                        \
  if (e == cudaSuccess) e = scan_set_attr<QB, NC>(smem_optin);
  ICC_SET(1, 1) ICC_SET(1, 2) ICC_SET(1, 3) ICC_SET(1, 4)
  ICC_SET(2, 1) ICC_SET(2, 2) ICC_SET(2, 3) ICC_SET(2, 4)
  ICC_SET(4, 1) ICC_SET(4, 2) ICC_SET(4, 3) ICC_SET(4, 4)
#undef ICC_SET
  if (e == cudaSuccess) e = cudaFuncSetAttribute(cluster_stream_topk_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(cluster_stream_topk_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(cluster_stream_topk_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(cluster_stream_topk_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  return e;
}

}  // namespace icc
