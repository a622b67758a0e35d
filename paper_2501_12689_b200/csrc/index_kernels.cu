// Two-level search (paper Sec. 4.1: cached examples clustered with K-Means into about sqrt(N)
// groups, a request matched to centroids first and searched inside the closest clusters).
// This file holds what is specific to it: the centroid seeding gather, the stable counting sort
// that turns row->cluster assignments into per-cluster member lists, the centroid update, and
// the scan of the probed clusters' rows with a fused partial top-k.  Scoring rows against
// centroids (assignment, and the centroid step of a query) runs on the ordinary scoring kernels.
#include <math.h>

#include "common.cuh"
#include "kernels.h"
#include "pipeline.cuh"

namespace icc {

// ------------------------------------------------------------------ seeding
// Centroid c starts as a copy of cache row slots[c]; its label is c.  One warp per centroid.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const __nv_bfloat16* __restrict__ slab, const int64_t* __restrict__ slots, int n_rows, int dim,
                   __nv_bfloat16* __restrict__ out_rows, int64_t* __restrict__ out_ids) {
  const int lane = threadIdx.x & 31;
  const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (c >= n_rows) return;
  const uint4* from = reinterpret_cast<const uint4*>(slab + slots[c] * dim);
  uint4* to = reinterpret_cast<uint4*>(out_rows + (int64_t)c * dim);
  for (int v = lane; v < (dim >> 3); v += 32) to[v] = from[v];
  if (lane == 0) out_ids[c] = c;
}

cudaError_t launch_gather_rows(const void* slab, const int64_t* slots, int n_rows, int dim, void* out_rows,
                               int64_t* out_ids, cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  gather_rows_kernel<<<(n_rows + 7) / 8, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(slab), slots, n_rows, dim,
                                                       static_cast<__nv_bfloat16*>(out_rows), out_ids);
  return cudaGetLastError();
}

// Cluster-contiguous copy of the indexed rows: row p of out_rows is cache row order[p], so the
// members of a cluster are one contiguous run that the two-level search streams.  One warp per row.
__global__ void __launch_bounds__(256)
gather_by_order_kernel(const __nv_bfloat16* __restrict__ slab, const int* __restrict__ order, int64_t n_rows, int dim,
                       __nv_bfloat16* __restrict__ out_rows) {
  const int lane = threadIdx.x & 31;
  const int64_t p = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (p >= n_rows) return;
  const uint4* from = reinterpret_cast<const uint4*>(slab + (int64_t)order[p] * dim);
  uint4* to = reinterpret_cast<uint4*>(out_rows + p * dim);
  for (int v = lane; v < (dim >> 3); v += 32) to[v] = ld_stream_16B(from + v);
}

cudaError_t launch_gather_by_order(const void* slab, const int* order, int64_t n_rows, int dim, void* out_rows,
                                   cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  gather_by_order_kernel<<<(unsigned)((n_rows + 7) / 8), 256, 0, st>>>(static_cast<const __nv_bfloat16*>(slab), order, n_rows,
                                                                        dim, static_cast<__nv_bfloat16*>(out_rows));
  return cudaGetLastError();
}

// ------------------------------------------------------------------ stable counting sort
// Rows are cut into blocks of SORT_ROWS_PER_BLOCK consecutive slots.
//   1. hist:    blk_hist[b][c] = rows of block b assigned to cluster c
//   2. prefix:  per cluster, exclusive prefix over the blocks (in place) and the cluster's total;
//               then the exclusive prefix over the clusters = offsets[K+1]
//   3. scatter: block b walks its rows in slot order and writes each to
//               order[offsets[c] + blk_hist[b][c] + rank among the block's earlier rows of c]
// so the members of every cluster end up in ascending slot order: the result does not depend on
// scheduling, which keeps the centroid sums and every later tie-break reproducible.
constexpr int SORT_ROWS_PER_BLOCK = 4096;

__global__ void __launch_bounds__(256)
sort_hist_kernel(const int64_t* __restrict__ assign, int64_t n, int n_clusters, int* __restrict__ blk_hist) {
  extern __shared__ int hist[];
  for (int c = threadIdx.x; c < n_clusters; c += blockDim.x) hist[c] = 0;
  __syncthreads();
  const int64_t r0 = (int64_t)blockIdx.x * SORT_ROWS_PER_BLOCK;
  const int64_t r1 = min(n, r0 + SORT_ROWS_PER_BLOCK);
  for (int64_t r = r0 + threadIdx.x; r < r1; r += blockDim.x) atomicAdd(&hist[(int)assign[r]], 1);
  __syncthreads();
  for (int c = threadIdx.x; c < n_clusters; c += blockDim.x) blk_hist[(size_t)blockIdx.x * n_clusters + c] = hist[c];
}

// One thread per cluster walks the blocks in order (reads of one step are coalesced over clusters).
__global__ void __launch_bounds__(256)
sort_prefix_blocks_kernel(int* __restrict__ blk_hist, int n_blocks, int n_clusters, int* __restrict__ totals) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n_clusters) return;
  int run = 0;
#pragma unroll 8
  for (int b = 0; b < n_blocks; ++b) {
    const size_t o = (size_t)b * n_clusters + c;
    const int v = blk_hist[o];
    blk_hist[o] = run;
    run += v;
  }
  totals[c] = run;
}

// Exclusive prefix over the cluster totals by one CTA: offsets[0] = 0 ... offsets[K] = n.
__global__ void __launch_bounds__(1024)
sort_prefix_clusters_kernel(const int* __restrict__ totals, int n_clusters, int* __restrict__ offsets) {
  __shared__ int warp_sum[32];
  __shared__ int carry;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int base = 0; base < n_clusters; base += 1024) {
    const int c = base + threadIdx.x;
    const int v = c < n_clusters ? totals[c] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(FULL_MASK, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = warp_sum[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL_MASK, w, o);
        if (lane >= o) w += t;
      }
      warp_sum[lane] = w;   // inclusive over warps
    }
    __syncthreads();
    const int before = carry + (warp > 0 ? warp_sum[warp - 1] : 0) + incl - v;
    if (c < n_clusters) offsets[c] = before;
    __syncthreads();
    if (threadIdx.x == 1023) carry = before + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) offsets[n_clusters] = carry;
}

// One warp per block of rows, 32 rows at a time in slot order.  Lanes that hold rows of the
// same cluster find each other with a match, rank themselves by lane and advance that
// cluster's cursor once.
__global__ void __launch_bounds__(32)
sort_scatter_kernel(const int64_t* __restrict__ assign, int64_t n, int n_clusters, const int* __restrict__ blk_hist,
                    const int* __restrict__ offsets, int* __restrict__ order) {
  extern __shared__ int cursor[];
  const int lane = threadIdx.x;
  for (int c = lane; c < n_clusters; c += 32) cursor[c] = offsets[c] + blk_hist[(size_t)blockIdx.x * n_clusters + c];
  __syncwarp();
  const int64_t r0 = (int64_t)blockIdx.x * SORT_ROWS_PER_BLOCK;
  const int64_t r1 = min(n, r0 + SORT_ROWS_PER_BLOCK);
  for (int64_t base = r0; base < r1; base += 32) {
    const int64_t r = base + lane;
    const bool live = r < r1;
    const int c = live ? (int)assign[r] : -1 - lane;   // dead lanes match nobody
    const unsigned peers = __match_any_sync(FULL_MASK, c);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    int at = 0;
    if (live) at = cursor[c];
    __syncwarp();
    if (live) {
      order[at + rank] = (int)r;
      if (rank == 0) cursor[c] = at + __popc(peers);
    }
    __syncwarp();
  }
}

static int g_sort_smem_limit = 48 * 1024;

cudaError_t index_configure(int smem_optin) {
  const int want = IC_INDEX_MAX_CLUSTERS * 4;
  if (want > smem_optin) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(sort_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, want);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(sort_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, want);
  if (e == cudaSuccess) g_sort_smem_limit = want;
  return e;
}

size_t sort_scratch_ints(int64_t n, int n_clusters) {
  const int64_t n_blocks = (n + SORT_ROWS_PER_BLOCK - 1) / SORT_ROWS_PER_BLOCK;
  return (size_t)n_blocks * n_clusters + (size_t)n_clusters;   // block histograms + totals
}

cudaError_t launch_sort_by_cluster(const int64_t* assign, int64_t n, int n_clusters, int* scratch, int* offsets,
                                   int* order, cudaStream_t st) {
  if (n <= 0 || n_clusters <= 0 || (size_t)n_clusters * 4 > (size_t)g_sort_smem_limit) return cudaErrorInvalidValue;
  const int n_blocks = (int)((n + SORT_ROWS_PER_BLOCK - 1) / SORT_ROWS_PER_BLOCK);
  int* blk_hist = scratch;
  int* totals = scratch + (size_t)n_blocks * n_clusters;
  const size_t smem = (size_t)n_clusters * 4;
  sort_hist_kernel<<<n_blocks, 256, smem, st>>>(assign, n, n_clusters, blk_hist);
  sort_prefix_blocks_kernel<<<(n_clusters + 255) / 256, 256, 0, st>>>(blk_hist, n_blocks, n_clusters, totals);
  sort_prefix_clusters_kernel<<<1, 1024, 0, st>>>(totals, n_clusters, offsets);
  sort_scatter_kernel<<<n_blocks, 32, smem, st>>>(assign, n, n_clusters, blk_hist, offsets, order);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ centroid update
// One CTA per cluster.  Thread t owns the dimension pairs t, t + 256, ...; it adds its components
// of the member rows in member-list (= slot) order into fp64 sums, so the sums are reproducible
// and equal to a sequential fp64 sum.  The centroid is the sum scaled to unit length, narrowed
// to fp32 and rounded to bf16; a cluster without rows (or whose rows cancel) keeps its centroid.
constexpr int UPD_THREADS = 256;
constexpr int UPD_MAX_PAIRS = 8;   // 256 threads * 8 pairs * 2 = 4096 = IC_MAX_DIM

__global__ void __launch_bounds__(UPD_THREADS)
centroid_update_kernel(const __nv_bfloat16* __restrict__ slab, int dim, const int* __restrict__ offsets,
                       const int* __restrict__ order, __nv_bfloat16* __restrict__ centroids) {
  __shared__ double red[UPD_THREADS / 32];
  __shared__ double norm_sh;
  const int c = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int m0 = offsets[c], m1 = offsets[c + 1];
  const int n_pairs = dim >> 1;
  double sx[UPD_MAX_PAIRS], sy[UPD_MAX_PAIRS];
#pragma unroll
  for (int t = 0; t < UPD_MAX_PAIRS; ++t) sx[t] = sy[t] = 0.0;
  const uint32_t* rows = reinterpret_cast<const uint32_t*>(slab);
  for (int m = m0; m < m1; m += 4) {
    // four member rows per step: their loads are issued together, their adds stay in order
    int64_t base[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) base[u] = (m + u < m1) ? (int64_t)order[m + u] * n_pairs : -1;
#pragma unroll
    for (int t = 0; t < UPD_MAX_PAIRS; ++t) {
      const int p = t * UPD_THREADS + tid;
      if (p < n_pairs) {
        uint32_t w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) w[u] = base[u] >= 0 ? rows[base[u] + p] : 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (base[u] >= 0) {
            sx[t] += (double)__uint_as_float(w[u] << 16);
            sy[t] += (double)__uint_as_float(w[u] & 0xffff0000u);
          }
        }
      }
    }
  }
  double ss = 0.0;
#pragma unroll
  for (int t = 0; t < UPD_MAX_PAIRS; ++t) ss += sx[t] * sx[t] + sy[t] * sy[t];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(FULL_MASK, ss, o);
  if (lane == 0) red[warp] = ss;
  __syncthreads();
  if (tid == 0) {
    double total = 0.0;
    for (int w = 0; w < UPD_THREADS / 32; ++w) total += red[w];
    norm_sh = sqrt(total);
  }
  __syncthreads();
  const double norm = norm_sh;
  if (m1 == m0 || !(norm > 0.0)) return;
  uint32_t* out = reinterpret_cast<uint32_t*>(centroids + (int64_t)c * dim);
#pragma unroll
  for (int t = 0; t < UPD_MAX_PAIRS; ++t) {
    const int p = t * UPD_THREADS + tid;
    if (p < n_pairs) {
      const __nv_bfloat16 lo = __float2bfloat16_rn(__double2float_rn(sx[t] / norm));
      const __nv_bfloat16 hi = __float2bfloat16_rn(__double2float_rn(sy[t] / norm));
      out[p] = (uint32_t)__bfloat16_as_ushort(lo) | ((uint32_t)__bfloat16_as_ushort(hi) << 16);
    }
  }
}

cudaError_t launch_centroid_update(const void* slab, int dim, const int* offsets, const int* order, int n_clusters,
                                   void* centroids, cudaStream_t st) {
  if (n_clusters <= 0) return cudaSuccess;
  centroid_update_kernel<<<n_clusters, UPD_THREADS, 0, st>>>(static_cast<const __nv_bfloat16*>(slab), dim, offsets, order,
                                                             static_cast<__nv_bfloat16*>(centroids));
  return cudaGetLastError();
}

// ------------------------------------------------------------------ scan of the probed clusters
// Work item (query q, list l).  Lists 0 .. n_probe*n_split-1 are the n_split pieces of the
// query's n_probe probed clusters (rows named by the cluster's member list); the remaining
// n_tail lists are pieces of the rows added after the clustering, [n_indexed, n), which every
// query searches.  One CTA per item: the query sits in shared memory as fp32, each warp takes
// every 8th group of four rows (four rows in flight per warp), lanes stride over the rows' 16-byte
// chunks, products are accumulated in fp32 and reduced by shuffles.  Each warp keeps a sorted
// candidate list of its own; at the end warp 0 merges the eight lists into the item's partial
// list partials[l][q][k].
constexpr int CS_WARPS = 8;
constexpr int CS_ROWS = 4;    // rows in flight per warp

__global__ void __launch_bounds__(CS_WARPS * 32)
cluster_scan_topk_kernel(const __nv_bfloat16* __restrict__ slab, const __nv_bfloat16* __restrict__ sorted_rows, int64_t n,
                         int dim, const float* __restrict__ q_f32, int nq, int k, const int64_t* __restrict__ probes,
                         int n_probe, int n_split, int n_tail, const int* __restrict__ offsets,
                         const int* __restrict__ order, int64_t n_indexed, uint64_t* __restrict__ partials, int l_begin) {
  extern __shared__ __align__(16) unsigned char cs_smem[];
  float* qs = reinterpret_cast<float*>(cs_smem);                         // [dim]
  uint64_t* lists = reinterpret_cast<uint64_t*>(qs + dim);               // [CS_WARPS][k]
  __shared__ uint64_t win_key[MAX_K];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_lists = n_probe * n_split + n_tail;
  const int lists_here = n_lists - l_begin;
  const int q = blockIdx.x / lists_here, l = l_begin + (blockIdx.x - q * lists_here);
  grid_dep_launch_dependents();
  grid_dep_wait();   // probes and the prepared query come from earlier kernels in the stream
  for (int j = tid; j < dim; j += CS_WARPS * 32) qs[j] = q_f32[(size_t)q * dim + j];
  for (int i = tid; i < CS_WARPS * k; i += CS_WARPS * 32) lists[i] = KEY_EMPTY;
  // the rows of this item: member-list positions [m0, m1), or slots [m0, m1) when order == nullptr
  int64_t m0 = 0, m1 = 0;
  const int* members = nullptr;
  if (l < n_probe * n_split) {
    const int64_t c = probes[(size_t)q * n_probe + l / n_split];
    if (c >= 0) {
      const int s = l % n_split;
      const int64_t o0 = offsets[c], len = offsets[c + 1] - o0;
      m0 = o0 + len * s / n_split;
      m1 = o0 + len * (s + 1) / n_split;
      members = order;
    }
  } else {
    const int t = l - n_probe * n_split;
    const int64_t len = n - n_indexed;
    m0 = n_indexed + len * t / n_tail;
    m1 = n_indexed + len * (t + 1) / n_tail;
  }
  __syncthreads();
  uint64_t* my_list = lists + (size_t)warp * k;
  uint64_t thr = KEY_EMPTY;
  const int n_chunks = dim >> 3;
  for (int64_t m = m0 + CS_ROWS * warp; m < m1; m += CS_ROWS * CS_WARPS) {
    // CS_ROWS rows per warp and step: all their loads are issued before the first product.  With a
    // cluster-contiguous copy of the rows the members of a cluster are read in place, one after
    // the other, and a row's slot is looked up in the member list only if its score can enter
    // the list; without one every row is fetched through the member list.
    int64_t pos[CS_ROWS];
    const uint4* row[CS_ROWS];
    float acc[CS_ROWS];
#pragma unroll
    for (int r = 0; r < CS_ROWS; ++r) {
      pos[r] = m + r < m1 ? m + r : m;   // a missing row repeats the first one and is dropped below
      const int64_t at = (members && !sorted_rows) ? (int64_t)members[pos[r]] : pos[r];
      row[r] = reinterpret_cast<const uint4*>(((members && sorted_rows) ? sorted_rows : slab) + at * dim);
      acc[r] = 0.0f;
    }
    for (int ch = lane; ch < n_chunks; ch += 32) {
      uint4 v[CS_ROWS];
#pragma unroll
      for (int r = 0; r < CS_ROWS; ++r) v[r] = ld_stream_16B(row[r] + ch);
      const float4 q0 = *reinterpret_cast<const float4*>(qs + 8 * ch);
      const float4 q1 = *reinterpret_cast<const float4*>(qs + 8 * ch + 4);
#pragma unroll
      for (int r = 0; r < CS_ROWS; ++r) {
        float x[8];
        bf16x8_to_f32(v[r], x);
        float a = acc[r];
        a = fmaf(x[0], q0.x, a);
        a = fmaf(x[1], q0.y, a);
        a = fmaf(x[2], q0.z, a);
        a = fmaf(x[3], q0.w, a);
        a = fmaf(x[4], q1.x, a);
        a = fmaf(x[5], q1.y, a);
        a = fmaf(x[6], q1.z, a);
        a = fmaf(x[7], q1.w, a);
        acc[r] = a;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
      for (int r = 0; r < CS_ROWS; ++r) acc[r] += __shfl_xor_sync(FULL_MASK, acc[r], o);
    }
#pragma unroll
    for (int r = 0; r < CS_ROWS; ++r) {
      if (m + r < m1 && score_to_ord(acc[r]) >= (uint32_t)(thr >> 32)) {   // warp-uniform (every lane holds the sum)
        const int64_t slot = members ? (int64_t)members[pos[r]] : pos[r];
        const uint64_t key = make_key(acc[r], (uint32_t)slot);
        if (key > thr) thr = warp_sorted_insert(my_list, k, key, lane);
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    const int r = tournament_in_registers<1>(lists, k, CS_WARPS, k, lane, win_key);
    __syncwarp();
    uint64_t* dst = partials + ((size_t)l * nq + q) * k;
    for (int i = lane; i < k; i += 32) dst[i] = i < r ? win_key[i] : KEY_EMPTY;
  }
}

cudaError_t launch_cluster_scan(const void* slab, const void* sorted_rows, int64_t n, int dim, const float* q_f32, int nq, int k,
                                const int64_t* probes, int n_probe, int n_split, int n_tail, const int* offsets,
                                const int* order, int64_t n_indexed, uint64_t* partials, int l_begin, cudaStream_t st) {
  const int n_lists = n_probe * n_split + n_tail;
  if (nq <= 0 || n_lists <= 0 || l_begin < 0 || l_begin > n_lists) return cudaErrorInvalidValue;
  if (l_begin == n_lists) return cudaSuccess;   // nothing left for this kernel
  const size_t smem = (size_t)dim * 4 + (size_t)CS_WARPS * k * 8;
  if (smem > 48 * 1024) return cudaErrorInvalidValue;
  return launch_overlapped(cluster_scan_topk_kernel, dim3((unsigned)(nq * (n_lists - l_begin))), dim3(CS_WARPS * 32), smem, st, 1,
                           static_cast<const __nv_bfloat16*>(slab), static_cast<const __nv_bfloat16*>(sorted_rows), n, dim,
                           q_f32, nq, k, probes, n_probe, n_split, n_tail, offsets, order, n_indexed, partials, l_begin);
}

}  // namespace icc
