// Host-side launchers of the library's kernels (internal to the shared library).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace icc {

// Launch `kernel` so that it may overlap the tail of the previous kernel in the stream
// (programmatic stream serialisation); cluster_x > 1 also asks for thread-block clusters.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     int cluster_x, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = (unsigned)n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Convert/normalise `nrows` input rows ([nrows, dim], fp32 if in_is_f32 else bf16) into bf16
// rows at out_bf16 (row pitch = dim elements).  Rows nrows .. pad_rows-1 of out_bf16 are set
// to zero.  If out_f32 != NULL it receives the stored bf16 values widened to fp32.
// ids_in/ids_out: optional, copies one int64 label per row alongside (used by insert).
cudaError_t launch_convert_rows(const void* in, int in_is_f32, int64_t nrows, int dim, int normalize,
                                void* out_bf16, float* out_f32, int64_t pad_rows, const int64_t* ids_in,
                                int64_t* ids_out, cudaStream_t st);

// Eviction support: slots whose id is in the sorted list `wanted` are appended (any order) to
// match_slots (capacity cap) and counted in *match_count (which may exceed cap).
cudaError_t launch_find_ids(const int64_t* ids, int64_t n, const int64_t* wanted, int64_t n_wanted, int64_t* match_slots,
                            unsigned long long* match_count, int64_t cap, cudaStream_t st);
// Move rows (and ids) inside the slab, src[i] -> dst[i]; the two sets must be disjoint.
// (utility: optional per-row fp32 side array that moves along.)
cudaError_t launch_move_rows(void* slab, int64_t* ids, float* utility, const int64_t* src, const int64_t* dst,
                             int64_t nmoves, int dim, cudaStream_t st);
// utility[row] += gains[j] for every j with wanted[j] == ids[row] (wanted sorted ascending; equal
// ids are added in their order); utility[row] *= factor for all rows.
cudaError_t launch_utility_add(const int64_t* ids, int64_t n, const int64_t* wanted, const float* gains, int64_t n_wanted,
                               float* utility, cudaStream_t st);
cudaError_t launch_utility_scale(float* utility, int64_t n, float factor, cudaStream_t st);

// Diagnostic: a bounded wait that is made to run out after limit_cycles (nothing completes the
// barrier); the kernel reports DEV_TIMEOUT_MBAR in the status word and returns.
cudaError_t launch_wait_limit_probe(long long limit_cycles, int* dev_status, cudaStream_t st);

// Generic CUDA-core scoring of up to 4 queries [q0, q0+4) against rows [0, n).
// partials: [n_part][nq][k] packed keys.
cudaError_t launch_generic(const void* slab, int64_t n, int dim, const float* q_f32, int q0, int nq,
                           int k, uint64_t* partials, int n_part, int smem_bytes, int* dev_status,
                           cudaStream_t st);

// Bulk-copy staged scan: qb in {1,2,4} queries starting at q0.
struct ScanParams {
  const void* slab;
  int64_t n;
  int dim;
  const float* q_f32;
  int q0, nq, qb, k;
  uint64_t* partials;
  int n_part;       // = number of CTAs
  int n_stages;
  int rows_per_stage;
  int smem_bytes;
  int* dev_status;
};
cudaError_t launch_scan(const ScanParams& p, cudaStream_t st);
cudaError_t scan_configure(int smem_optin);

// tcgen05 scoring: query tiles of 128 (or one resident tile of 64) x row tiles of 256, top-k fused
// in the epilogue.
constexpr int PACE_EVERY = 4;   // a CTA publishes and compares its progress at every PACE_EVERY-th row tile
struct UmmaParams {
  CUtensorMap tmap_q;     // [nq_pad, dim] bf16, box 64 x 128 (64 x 64 with q_resident), 128-byte swizzle
  CUtensorMap tmap_slab;  // [capacity, dim] bf16, box 64 x 256, 128-byte swizzle
  CUtensorMap tmap_slab_half;  // same tensor, box 64 x 128 (CTA pairs and resident queries)
  int cta_group;          // 1, or 2 = CTA pairs sharing each row tile
  int q_resident;         // 1: at most 64 queries, M = 64, the query tile stays in shared memory
  int64_t n;
  int64_t tile_begin, tile_end;   // 256-row tiles scored by this launch
  int dim;
  int nq, k;
  const uint64_t* thr_floor;      // optional [nq] keys: candidates at or below are discarded
  int n_query_tiles;
  int n_part;
  int n_stages;
  int queue_cap;          // per-query candidate queue entries in shared memory
  int smem_bytes;
  uint64_t* partials;     // [n_part][nq][k]
  unsigned long long* pace;   // optional [n_part][units per partition] progress words (L2 pacing hint)
  unsigned epoch;             // number of this launch, unique in the process: tells this launch's progress
                              // words and seeding flags from older ones
  int pace_window;            // tiles a CTA may be ahead of the slowest published progress (>= PACE_EVERY + 2)
  float* seed_maxima;         // optional [n_query_tiles][n_part][seed_t0][128][4]: seeding inside the launch (needs
  unsigned* seed_flags;       // thr_floor == NULL and full first tiles); flags [n_query_tiles][n_part][4]
  int seed_look_cycles;       // longest an epilogue warp looks for its siblings' maxima, in SM cycles
  int seed_t0;                // tiles per CTA whose group maxima are exchanged (the first seed_t0 - 1 of them
                              // are visited for their maxima only and scored at the end of the launch)
  int* dev_status;
};
cudaError_t launch_umma(const UmmaParams& p, cudaStream_t st);
// Dynamic shared memory a launch of that shape needs.
size_t umma_smem_bytes(int cta_group, bool q_resident, int dim, int k, int queue_cap, int n_stages);
cudaError_t umma_configure(int smem_optin);

// Merge n_part partial lists per query into the final sorted top-k and gather ids.  Entries
// scoring below min_score (-inf: none) are reported as absent; out_counts (optional, [nq])
// receives the number of entries kept per query.
cudaError_t launch_merge(const uint64_t* partials, int n_part, int nq, int k, const int64_t* ids,
                         int64_t* out_ids, float* out_scores, float min_score, int32_t* out_counts,
                         cudaStream_t st, int64_t self_slot0 = -1);
// self_slot0 >= 0: query q is cache row self_slot0 + q; out_ids/out_scores then hold ONE entry
// per query, the best-scoring entry other than that row.
// Same merge, but the result stays in key form: out_keys [nq][k] (sorted, KEY_EMPTY padded)
// and out_thr [nq] = the k-th key (KEY_EMPTY when fewer than k candidates exist).
cudaError_t launch_merge_keys(const uint64_t* partials, int n_part, int nq, int k, uint64_t* out_keys,
                              uint64_t* out_thr, cudaStream_t st);
cudaError_t merge_configure(int smem_optin);

// Two-level search, pieces of probed clusters streamed from the cluster-contiguous copy of the rows
// (scan_kernel.cu; dim <= 1024).  One CTA per (query, probe, piece); partials as for launch_cluster_scan.
struct ClusterStreamParams {
  const void* sorted_rows;   // row p = cache row order[p]
  int dim;
  const float* q_f32;
  int nq, k;
  const int64_t* probes;     // [nq][n_probe], -1 = none
  int n_probe, n_split;
  const int* offsets;
  const int* order;
  uint64_t* partials;        // [n_probe * n_split (+ lists of other kernels)][nq][k]
  int n_stages;
  int smem_bytes;
  int* dev_status;
};
cudaError_t launch_cluster_stream(const ClusterStreamParams& p, cudaStream_t st);
int cluster_stream_smem_bytes(int dim, int k, int n_stages);

// ---- two-level search (index_kernels.cu)
constexpr int IC_INDEX_MAX_CLUSTERS = 16384;   // must equal IC_MAX_CLUSTERS; bounds the sort kernels' shared memory
cudaError_t index_configure(int smem_optin);
// Rows slots[c] of the slab become rows c of out_rows, labelled c.
cudaError_t launch_gather_rows(const void* slab, const int64_t* slots, int n_rows, int dim, void* out_rows,
                               int64_t* out_ids, cudaStream_t st);
// Stable counting sort of rows 0 .. n-1 by assign[row] in [0, n_clusters): offsets[n_clusters+1]
// and order[n] (members of cluster c are order[offsets[c] .. offsets[c+1]), ascending slots).
// scratch must hold sort_scratch_ints(n, n_clusters) ints.
size_t sort_scratch_ints(int64_t n, int n_clusters);
cudaError_t launch_sort_by_cluster(const int64_t* assign, int64_t n, int n_clusters, int* scratch, int* offsets,
                                   int* order, cudaStream_t st);
// Centroid c (row c of centroids, bf16) becomes the unit-length mean of its member rows.
cudaError_t launch_centroid_update(const void* slab, int dim, const int* offsets, const int* order, int n_clusters,
                                   void* centroids, cudaStream_t st);
// Row p of out_rows becomes cache row order[p] (the cluster-contiguous copy the two-level search streams).
cudaError_t launch_gather_by_order(const void* slab, const int* order, int64_t n_rows, int dim, void* out_rows,
                                   cudaStream_t st);
// Scores, per query, the rows of its n_probe probed clusters (probes [nq][n_probe], -1 = none),
// each cut into n_split pieces, and the rows [n_indexed, n) cut into n_tail pieces; writes one
// sorted partial list per piece: partials [n_probe*n_split + n_tail][nq][k].
// sorted_rows (optional): rows of the indexed slots in member-list order (row p = cache row order[p]).
// l_begin: first list this launch produces (n_probe * n_split when another kernel scans the clusters).
cudaError_t launch_cluster_scan(const void* slab, const void* sorted_rows, int64_t n, int dim, const float* q_f32, int nq, int k,
                                const int64_t* probes, int n_probe, int n_split, int n_tail, const int* offsets,
                                const int* order, int64_t n_indexed, uint64_t* partials, int l_begin, cudaStream_t st);

}  // namespace icc
