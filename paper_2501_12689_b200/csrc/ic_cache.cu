// Host side of the C ABI declared in include/ic_cache.h: argument checking, buffer ownership,
// launch planning and kernel sequencing.  All arithmetic of the retrieval path runs in the
// kernels; nothing here touches embedding data on the CPU.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <atomic>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/ic_cache.h"
#include "kernels.h"

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof g_err, fmt, ap);
  va_end(ap);
  return code;
}

constexpr int WINDOW_MAX_NQ = 1024;   // queries scored per pass over the slab
constexpr int QUERY_TILE = 128;       // tcgen05 path: queries per CTA (MMA M)
constexpr int ROW_TILE = 256;         // tcgen05 path: cache rows per accumulator (MMA N)
constexpr int K_CHUNK = 64;           // tcgen05 path: bf16 elements per 128-byte swizzled row
constexpr int RESIDENT_MAX_NQ = 64;   // tcgen05 path: batches up to this size keep their query tile in shared memory
constexpr int RESIDENT_MIN_STAGES = 4;
constexpr int SCAN_MAX_Q = 4;        // queries per scan launch
constexpr int SCAN_AUTO_MAX_Q = 2;   // largest batch the automatic choice gives to the scan path
constexpr int SCAN_MAX_DIM = 1024;
constexpr int SCAN_AUTO_MIN_DIM = 512;   // shorter rows go to the tensor-core path even for one query
constexpr int SCAN_ROWS_PER_STAGE = 32;
constexpr int SCAN_CONSUMER_WARPS = 8;
constexpr int GENERIC_QB = 4;
constexpr int SEED_MIN_TILES_PER_CTA = 8;  // tcgen05 path: seed thresholds when a CTA has this many tiles
constexpr int SEED_FRACTION = 16;          // share of the row tiles scored by the seeding pass
constexpr int SEED_TWO_LEVEL_TILES_PER_CTA = 4;
constexpr int64_t DENSE_TAIL_MIN_ROWS = 1024;   // two-level search: rows past the index from which they go to the tensor-core kernel
// Words that the CTAs of one tensor-core launch exchange: 8 KiB of progress words (L2 pacing, one per
// CTA or pair) followed by 8 KiB of seeding flags (one per CTA).  Every word carries the launch's
// number, drawn from one counter for the whole process, so words of earlier launches (of any handle
// that shares the block) are never taken for current ones.
constexpr size_t PACE_BYTES = 16384;
constexpr size_t SEED_FLAGS_OFFSET = 8192;
std::atomic<unsigned> g_launch_epoch{0};
unsigned next_epoch() {
  unsigned e = ++g_launch_epoch;
  if (e == 0) e = ++g_launch_epoch;   // 0 is what a cleared word holds
  return e;
}

struct DeviceGuard {
  int prev = -1;
  bool changed = false;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) changed = (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() {
    if (changed) cudaSetDevice(prev);
  }
};

struct Buffer {
  void* p = nullptr;
  size_t bytes = 0;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

}  // namespace

struct ic_cache {
  int device = 0;
  int dim = 0;
  int64_t capacity = 0;
  int64_t size = 0;
  int input_dtype = IC_BF16;
  int normalize = 0;
  int forced_path = IC_PATH_AUTO;
  int sm_count = 0;
  int smem_optin = 0;
  cudaStream_t stream = nullptr;
  void* slab = nullptr;
  bool own_slab = false;
  int64_t* ids = nullptr;
  bool own_ids = false;
  Buffer q_bf16, q_f32, partials, thr, maxima, pace, stage_in, stage_ids, stage_scores, evict;
  int l2_bytes = 0;
  int* h_status = nullptr;  // pinned, mapped; kernels write a code when a bounded wait expires
  int* d_status = nullptr;
  int64_t launches = 0;
  // two-level search: the centroids live in a child cache (labels 0 .. n_clusters-1) so that the
  // ordinary scoring kernels serve both the assignment step and a query's centroid step
  ic_cache* centroids = nullptr;
  int32_t n_clusters = 0;
  int64_t n_indexed = 0;
  unsigned char* workspace = nullptr;   // optional caller-owned scratch for ic_cache_query (borrowed)
  size_t workspace_bytes = 0;
  float* utility = nullptr;   // [capacity] per-entry utility, allocated on first use, zero for new entries
  Buffer util_ids, util_gains;
  Buffer idx_assign, idx_best, idx_order, idx_offsets, idx_sort, idx_init, idx_probes, idx_probe_scores;
  Buffer idx_rows;            // cluster-contiguous copy of the indexed rows (optional: absent if memory is short)
  bool have_idx_rows = false;
  EncodeTiledFn encode = nullptr;
  CUtensorMap tmap_slab;       // box of 256 rows
  CUtensorMap tmap_slab_half;  // box of 128 rows, for CTA pairs
  bool have_tmap_slab = false;
  // optional per-kernel timing (ic_cache_set_profiling)
  bool profiling = false;
  std::vector<cudaEvent_t> ev_score, ev_merge, ev_seed;   // start/stop pairs
  size_t n_ev_score = 0, n_ev_merge = 0, n_ev_seed = 0;   // events used since the last read
};

namespace {

size_t in_elem_bytes(const ic_cache* c) { return c->input_dtype == IC_F32 ? 4 : 2; }

bool is_device_ptr(const void* p, int device) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
    cudaGetLastError();
    return false;
  }
  if (a.type == cudaMemoryTypeManaged) return true;
  return a.type == cudaMemoryTypeDevice && a.device == device;
}

int ensure(ic_cache* c, Buffer& b, size_t bytes, const char* what) {
  if (bytes <= b.bytes) return IC_OK;
  if (b.p) {
    // the old buffer may still be in use by enqueued work
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(IC_ERR_CUDA, "stream sync failed while growing %s", what);
    cudaFree(b.p);
    b.p = nullptr;
    b.bytes = 0;
  }
  cudaError_t e = cudaMalloc(&b.p, bytes);
  if (e != cudaSuccess) {
    cudaGetLastError();
    b.p = nullptr;
    return fail(IC_ERR_NOMEM, "cudaMalloc of %zu bytes for %s failed: %s", bytes, what, cudaGetErrorString(e));
  }
  b.bytes = bytes;
  return IC_OK;
}

void release(Buffer& b) {
  if (b.p) cudaFree(b.p);
  b.p = nullptr;
  b.bytes = 0;
}

int encode_2d(ic_cache* c, CUtensorMap* tm, const void* base, uint64_t rows, uint32_t box_rows) {
  // [rows, dim] bf16 row-major; box = K_CHUNK elements (128 bytes) x box_rows rows, 128-byte
  // swizzle; out-of-range elements (row tail, dim tail) read as zero.
  cuuint64_t dims[2] = {(cuuint64_t)c->dim, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)c->dim * 2};
  cuuint32_t box[2] = {(cuuint32_t)K_CHUNK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = c->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                         estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(IC_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return IC_OK;
}

int plan_impl(int32_t dim, int64_t n, int32_t nq, int32_t k, int32_t path, int32_t sm_count,
              int32_t smem_optin, ic_cache_plan_t* out) {
  if (!out) return fail(IC_ERR_INVALID, "plan: NULL output");
  memset(out, 0, sizeof *out);
  if (dim < 8 || dim > IC_MAX_DIM || (dim % 8) != 0) return fail(IC_ERR_INVALID, "dim %d must be a multiple of 8 in [8, %d]", dim, IC_MAX_DIM);
  if (n < 0 || nq < 1 || k < 1 || k > IC_MAX_K) return fail(IC_ERR_INVALID, "plan: need n >= 0, nq >= 1, 1 <= k <= %d", IC_MAX_K);
  if (sm_count < 1 || smem_optin < 48 * 1024) return fail(IC_ERR_INVALID, "plan: bad device limits");
  if (path < IC_PATH_AUTO || path > IC_PATH_UMMA) return fail(IC_ERR_INVALID, "plan: unknown path %d", path);
  const int window = std::min<int>(nq, WINDOW_MAX_NQ);
  const int n_windows = (nq + WINDOW_MAX_NQ - 1) / WINDOW_MAX_NQ;
  // measured crossover (N = 1 M, d = 768, k = 10): the scan wins for one or two queries, the
  // tensor-core path from three on (its time hardly grows with nq while HBM-bound)
  // (and only for rows of at least 1 KiB: at dim = 384, N = 2 M, one query takes 271 us on the scan
  // against 245 us on the tensor-core path; at dim = 768 and 1024 the scan is 2-4 % ahead in long runs)
  if (path == IC_PATH_AUTO)
    path = (nq <= SCAN_AUTO_MAX_Q && dim <= SCAN_MAX_DIM && dim >= SCAN_AUTO_MIN_DIM) ? IC_PATH_SCAN : IC_PATH_UMMA;
  out->path = path;
  const int merge_lists_max = (smem_optin - 4096) / (k * 8 + 4);
  if (path == IC_PATH_GENERIC) {
    out->query_tile = GENERIC_QB;
    out->n_query_tiles = (window + GENERIC_QB - 1) / GENERIC_QB;
    out->n_partitions = std::max(1, std::min(2 * sm_count, merge_lists_max));
    out->n_ctas = out->n_partitions;
    out->n_stages = 0;
    out->smem_bytes = GENERIC_QB * k * 8 + 64;
    out->n_launches = n_windows * out->n_query_tiles;
  } else if (path == IC_PATH_SCAN) {
    if (dim > SCAN_MAX_DIM) return fail(IC_ERR_UNSUPPORTED, "scan path needs dim <= %d", SCAN_MAX_DIM);
    out->query_tile = window <= 1 ? 1 : (window <= 2 ? 2 : SCAN_MAX_Q);
    out->n_query_tiles = (window + out->query_tile - 1) / out->query_tile;
    out->n_partitions = std::max(1, std::min(sm_count, merge_lists_max));
    out->n_ctas = out->n_partitions;
    const int stage_bytes = SCAN_ROWS_PER_STAGE * dim * 2;
    const int fixed = 2048 + SCAN_CONSUMER_WARPS * SCAN_MAX_Q * k * 8;   // header + per-warp lists
    out->n_stages = std::min(8, (smem_optin - fixed) / stage_bytes);
    if (out->n_stages < 2) return fail(IC_ERR_UNSUPPORTED, "scan path: shared memory too small for dim %d", dim);
    out->smem_bytes = fixed + out->n_stages * stage_bytes;
    out->n_launches = n_windows * out->n_query_tiles;
  } else {
    out->query_tile = QUERY_TILE;
    out->n_query_tiles = (window + QUERY_TILE - 1) / QUERY_TILE;
    // An even number of query tiles runs as CTA pairs (one 256-query MMA per pair): each CTA
    // then stages only half of every row tile.
    out->cta_group = (out->n_query_tiles % 2 == 0 && sm_count >= 2) ? 2 : 1;
    if (const char* env = getenv("IC_CACHE_CTA_GROUP")) {   // tuning knob: "1" forces single CTAs
      if (env[0] == '1' && env[1] == 0) out->cta_group = 1;
    }
    const int units = out->n_query_tiles / out->cta_group;                    // CTAs or pairs per partition
    out->n_partitions = std::max(1, std::min((sm_count / out->cta_group) / units, merge_lists_max - 1));
    out->n_ctas = out->n_partitions * out->n_query_tiles;
    // Threshold seeding, with enough row tiles per CTA.  Level 0 (seed0_tiles, about one tile per
    // SM) happens inside the scoring launch: every CTA publishes the group maxima of its first
    // tiles and takes, per query, (about) the k-th largest of all of them as a floor.  Level 1
    // (seed_tiles, large caches only): 1/16 of the tiles are scored first, by a launch of their
    // own, into real lists, whose merge gives the sample's exact k-th key as the floor of the
    // main pass, which then skips the sampled tiles.
    const int64_t n_tiles = (n + ROW_TILE - 1) / ROW_TILE;
    const char* seed_env = getenv("IC_CACHE_SEED");   // tuning knob: "0" scores everything in one pass, unseeded
    const bool seeding = !(seed_env && seed_env[0] == '0' && seed_env[1] == 0);
    const int P = out->n_partitions;
    if (seeding && n_tiles >= (int64_t)SEED_MIN_TILES_PER_CTA * P) {
      int seed_fraction = SEED_FRACTION;
      if (const char* fe = getenv("IC_CACHE_SEED_FRACTION")) {   // tuning knob: 1/fraction of the tiles are sampled
        const int f = atoi(fe);
        if (f >= 2) seed_fraction = f;
      }
      const int64_t t = n_tiles / seed_fraction / P * P;
      if (t >= (int64_t)SEED_TWO_LEVEL_TILES_PER_CTA * P && t > P) out->seed_tiles = (int32_t)t;
      // tiles per CTA whose maxima are exchanged inside the (first) launch: about one tile per SM
      // in all, so that the sample does not shrink when there are few partitions
      const int64_t first_launch_tiles = out->seed_tiles > 0 ? out->seed_tiles : n / ROW_TILE;   // full tiles only
      int64_t t0 = std::min<int64_t>({(sm_count + P - 1) / P, 16, first_launch_tiles / P});
      // A sampling launch of a batch of several query tiles (tensor-bound) starts from a floor that
      // a few hundred candidates per query still pass, and its epilogue, unlike the main pass's, is
      // then slower than its MMAs.  Up to a ninth of its tiles (at most 24 per CTA) go into the first
      // floor instead: visiting them twice costs less than the admissions it saves (measured at
      // 16 M x 768: sampling launch 2.2 -> 1.9 ms for 1024 queries, 1.26 -> 1.07 ms for 512).
      if (out->seed_tiles > 0 && out->n_query_tiles >= 2)
        t0 = std::max<int64_t>(t0, std::min<int64_t>(24, first_launch_tiles / P / 9));
      if (t0 >= 1 && t0 * P * 4 >= k) out->seed0_tiles = (int32_t)(t0 * P);
      else out->seed_tiles = 0;   // no first floor: the sample launch would start cold
    }
    // Shared memory: as many candidate queue entries per query (up to 8) as still leave room for the
    // smallest ring, then as many ring stages as fit.  Batches of at most 64 queries keep their whole
    // query tile resident (M = 64) when that still leaves a ring of four 16 KiB stages.
    int max_stages = 12;
    if (const char* env = getenv("IC_CACHE_MAX_STAGES")) {   // tuning knob: cap on the ring depth
      const int cap = atoi(env);
      if (cap >= 2) max_stages = std::min(max_stages, cap);
    }
    auto fit = [&](bool resident, int min_stages, int* qcap, int* stages) {
      for (int qc = 8; qc >= 1; --qc) {
        if (icc::umma_smem_bytes(out->cta_group, resident, dim, k, qc, min_stages) > (size_t)smem_optin) continue;
        int st = min_stages;
        while (st < max_stages && icc::umma_smem_bytes(out->cta_group, resident, dim, k, qc, st + 1) <= (size_t)smem_optin) ++st;
        *qcap = qc;
        *stages = st;
        return true;
      }
      return false;
    };
    const char* qres_env = getenv("IC_CACHE_QRES");   // tuning knob: "0" streams the query tile for every batch size
    const bool want_resident = window <= RESIDENT_MAX_NQ && !(qres_env && qres_env[0] == '0' && qres_env[1] == 0);
    int qcap = 0, stages = 0;
    if (want_resident && fit(true, std::min(RESIDENT_MIN_STAGES, max_stages), &qcap, &stages)) {
      out->query_resident = 1;
      out->query_tile = RESIDENT_MAX_NQ;
    } else if (!fit(false, 2, &qcap, &stages)) {
      return fail(IC_ERR_UNSUPPORTED, "tensor-core path: shared memory too small");
    }
    // twice the queue (fewer drains) when it costs no ring stage
    if (qcap == 8 && icc::umma_smem_bytes(out->cta_group, out->query_resident != 0, dim, k, 16, stages) <= (size_t)smem_optin) qcap = 16;
    out->queue_cap = qcap;
    out->n_stages = stages;
    out->smem_bytes = (int32_t)icc::umma_smem_bytes(out->cta_group, out->query_resident != 0, dim, k, qcap, stages);
    out->n_launches = n_windows * (1 + (out->seed_tiles > 0 ? 1 : 0));
  }
  return IC_OK;
}

constexpr size_t MAX_PROFILE_EVENTS = 2 * 16384;

// Record one event of a start/stop pair; silently stops recording when the pool is full.
void profile_mark(ic_cache* c, std::vector<cudaEvent_t>& pool, size_t& used) {
  if (!c->profiling || used >= MAX_PROFILE_EVENTS) return;
  if (used == pool.size()) {
    cudaEvent_t ev;
    if (cudaEventCreate(&ev) != cudaSuccess) {
      cudaGetLastError();
      return;
    }
    pool.push_back(ev);
  }
  cudaEventRecord(pool[used++], c->stream);
}

int check_timeout(ic_cache* c) {
  if (c->h_status && *reinterpret_cast<volatile int*>(c->h_status) != 0)
    return fail(IC_ERR_TIMEOUT, *c->h_status == 3 ? "an earlier kernel failed a debug-build index check (code %d); call ic_cache_sync to clear"
                                                  : "an earlier kernel gave up on a bounded wait (code %d); call ic_cache_sync to clear", *c->h_status);
  return IC_OK;
}

int do_insert(ic_cache* c, const void* emb, const int64_t* ids, int64_t n) {
  cudaError_t e = icc::launch_convert_rows(emb, c->input_dtype == IC_F32, n, c->dim, c->normalize,
                                           static_cast<char*>(c->slab) + (size_t)c->size * c->dim * 2, nullptr, n, ids,
                                           c->ids + c->size, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "insert kernel launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  if (c->utility) {   // new entries start without utility
    if (cudaMemsetAsync(c->utility + c->size, 0, (size_t)n * 4, c->stream) != cudaSuccess)
      return fail(IC_ERR_CUDA, "clearing the new entries' utility failed");
  }
  c->size += n;
  return IC_OK;
}

// The utility side array exists from the first call that needs it; until then every utility is 0.
int ensure_utility(ic_cache* c) {
  if (c->utility) return IC_OK;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&c->utility), (size_t)c->capacity * 4);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->utility, 0, (size_t)c->capacity * 4, c->stream);
  if (e != cudaSuccess) {
    cudaGetLastError();
    if (c->utility) cudaFree(c->utility);
    c->utility = nullptr;
    return fail(IC_ERR_NOMEM, "allocation of the utility array (%zu bytes) failed: %s", (size_t)c->capacity * 4, cudaGetErrorString(e));
  }
  return IC_OK;
}

// Bytes of group maxima that seeding inside a tensor-core launch exchanges: four floats per
// (query tile, partition, tensor-memory lane).
size_t seed_maxima_bytes(const ic_cache_plan_t& pl) {
  return (size_t)pl.n_query_tiles * pl.seed0_tiles * QUERY_TILE * 16;
}

// Tensor-core scoring of one window.  Large caches: a launch over the first seed_tiles tiles into
// real lists, whose merge gives the sample's exact k-th key per query as the floor of the main
// pass; then the main pass over the tiles not yet in a list.  A launch that is given no floors
// seeds itself from the group maxima of its CTAs' first tiles (seed0_tiles > 0).  Lists are blocks
// of nq*k keys inside `partials`:
//   blocks 0 .. P-1      main pass            block P          merged sample list
//   blocks P+1 .. 2P     lists of the sampling launch
// On return *n_final_lists tells the final merge how many leading blocks to read.
int run_umma_passes(ic_cache* c, const ic_cache_plan_t& pl, const void* q_bf16, int nq, int nq_pad, int k,
                    uint64_t* partials, uint64_t* thr, float* maxima, unsigned long long* pace, int* n_final_lists,
                    bool profile, int64_t only_from_tile = -1) {
  if (!c->have_tmap_slab) return fail(IC_ERR_UNSUPPORTED, "tensor-core path unavailable: no tensor map for the slab");
  const int P = pl.n_partitions;
  const size_t list_block = (size_t)nq * k;
  icc::UmmaParams up;
  int rc = encode_2d(c, &up.tmap_q, q_bf16, (uint64_t)nq_pad, pl.query_resident ? RESIDENT_MAX_NQ : QUERY_TILE);
  if (rc != IC_OK) return rc;
  up.tmap_slab = c->tmap_slab;
  up.tmap_slab_half = c->tmap_slab_half;
  up.cta_group = pl.cta_group;
  up.q_resident = pl.query_resident;
  up.n = c->size;
  up.dim = c->dim;
  up.nq = nq;
  up.k = k;
  up.n_query_tiles = pl.n_query_tiles;
  up.n_part = P;
  up.n_stages = pl.n_stages;
  up.queue_cap = pl.queue_cap;
  up.smem_bytes = pl.smem_bytes;
  up.dev_status = c->d_status;
  up.seed_t0 = pl.seed0_tiles / P;
  up.seed_look_cycles = 60000;   // ~30 us
  if (const char* env = getenv("IC_CACHE_SEED_LOOK_CYCLES")) {   // tuning and test knob: 0 = never wait for the siblings
    const int v = atoi(env);
    if (v >= 0) up.seed_look_cycles = v;
  }
  // CTAs of one partition may run half of the partition's share of L2 apart.  Progress is published
  // at every PACE_EVERY-th tile only, so a word can be that stale (siblings in step still look
  // PACE_EVERY apart) and a CTA moves on as many tiles between two looks: the window is what is left
  // of the half share, and never less than the staleness plus some jitter.
  up.pace = pace;
  const int64_t tile_bytes = (int64_t)ROW_TILE * c->dim * 2;
  up.pace_window = (int)std::max<int64_t>(icc::PACE_EVERY + 2,
      std::min<int64_t>(32, (int64_t)c->l2_bytes / 2 / ((int64_t)P * tile_bytes) - icc::PACE_EVERY));
  if (const char* env = getenv("IC_CACHE_PACE_WINDOW")) {   // tuning knob: tiles; 0 switches pacing off
    const int w = atoi(env);
    if (w <= 0) up.pace = nullptr;
    else up.pace_window = w;
  }
  const int64_t n_tiles = (c->size + ROW_TILE - 1) / ROW_TILE;
  uint64_t* pass_lists = partials + (size_t)(P + 1) * list_block;
  uint64_t* merged = partials + (size_t)P * list_block;
  // only_from_tile >= 0: a single launch over the tiles from there on, no seeding (the two-level
  // search uses it for the rows inserted after its index was built)
  const bool whole = only_from_tile < 0;
  // seeding inside a launch: its flags sit behind the progress words
  const bool self_seed = whole && pl.seed0_tiles > 0 && maxima != nullptr && pace != nullptr;
  unsigned* flags = reinterpret_cast<unsigned*>(reinterpret_cast<unsigned char*>(pace) + SEED_FLAGS_OFFSET);
  bool have_thr = false;
  int64_t begin = whole ? 0 : only_from_tile;
  *n_final_lists = P;
  cudaError_t e;
  if (whole && pl.seed_tiles > 0) {
    up.tile_begin = 0;
    up.tile_end = pl.seed_tiles;
    up.thr_floor = nullptr;
    up.partials = pass_lists;
    up.seed_maxima = self_seed ? maxima : nullptr;
    up.seed_flags = self_seed ? flags : nullptr;
    up.epoch = next_epoch();
    if (profile) profile_mark(c, c->ev_seed, c->n_ev_seed);
    e = icc::launch_umma(up, c->stream);
    if (e != cudaSuccess) return fail(IC_ERR_CUDA, "tensor-core sampling launch failed: %s", cudaGetErrorString(e));
    c->launches += 1;
    e = icc::launch_merge_keys(pass_lists, P, nq, k, merged, thr, c->stream);
    if (e != cudaSuccess) return fail(IC_ERR_CUDA, "sample merge launch failed: %s", cudaGetErrorString(e));
    c->launches += 1;
    if (profile) profile_mark(c, c->ev_seed, c->n_ev_seed);
    have_thr = true;
    begin = pl.seed_tiles;
    *n_final_lists = P + 1;
  }
  up.tile_begin = begin;
  up.tile_end = n_tiles;
  up.thr_floor = have_thr ? thr : nullptr;
  up.partials = partials;
  up.seed_maxima = (self_seed && !have_thr) ? maxima : nullptr;
  up.seed_flags = (self_seed && !have_thr) ? flags : nullptr;
  up.epoch = next_epoch();
  if (profile) profile_mark(c, c->ev_score, c->n_ev_score);
  e = icc::launch_umma(up, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "tensor-core scoring launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  if (profile) profile_mark(c, c->ev_score, c->n_ev_score);
  return IC_OK;
}

// One window of at most WINDOW_MAX_NQ queries, all pointers on the device.
int do_query_window(ic_cache* c, const void* q, int nq, int k, int64_t* out_ids, float* out_scores, float min_score,
                    int32_t* out_counts) {
  ic_cache_plan_t pl;
  int rc = plan_impl(c->dim, c->size, nq, k, c->forced_path, c->sm_count, c->smem_optin, &pl);
  if (rc != IC_OK) return rc;
  const int nq_pad = (nq + QUERY_TILE - 1) / QUERY_TILE * QUERY_TILE;
  if ((rc = ensure(c, c->q_bf16, (size_t)nq_pad * c->dim * 2, "query staging (bf16)")) != IC_OK) return rc;
  if ((rc = ensure(c, c->q_f32, (size_t)nq * c->dim * 4, "query staging (fp32)")) != IC_OK) return rc;
  // lists of the main pass, two merged sample lists, lists of a seeding pass
  const size_t list_block = (size_t)nq * k;   // keys of one partition
  if ((rc = ensure(c, c->partials, (size_t)(2 * pl.n_partitions + 2) * list_block * 8, "partial top-k lists")) != IC_OK) return rc;
  if ((rc = ensure(c, c->thr, (size_t)nq * 8, "seed thresholds")) != IC_OK) return rc;
  if ((rc = ensure(c, c->maxima, seed_maxima_bytes(pl), "group maxima")) != IC_OK) return rc;

  // bf16 queries that need no normalisation go to the tensor-core path as they are: the query
  // tensor map points at the caller's rows and rows past nq read as zero, so the conversion
  // launch (and its place in the chain of dependent kernels) is saved.  With a streamed query
  // tile only when its last 128 rows are nearly all there: out-of-range rows load slowly, and
  // they would be loaded with every ring stage (measured main pass, 500-step runs: 64 queries
  // 240 -> 262 us, 16 queries 221 -> 261 us; 100 and 128 queries unchanged, step 2-4 us shorter).
  // A resident query tile is loaded once per CTA, so there it always pays.
  const bool direct = pl.path == IC_PATH_UMMA && c->input_dtype == IC_BF16 && !c->normalize &&
                      (reinterpret_cast<uintptr_t>(q) & 15) == 0 &&
                      (pl.query_resident || nq_pad - nq <= QUERY_TILE / 4);
  cudaError_t e = cudaSuccess;
  if (!direct) {
    e = icc::launch_convert_rows(q, c->input_dtype == IC_F32, nq, c->dim, c->normalize, c->q_bf16.p,
                                 static_cast<float*>(c->q_f32.p), nq_pad, nullptr, nullptr, c->stream);
    if (e != cudaSuccess) return fail(IC_ERR_CUDA, "query preparation launch failed: %s", cudaGetErrorString(e));
    c->launches += 1;
  }
  uint64_t* partials = static_cast<uint64_t*>(c->partials.p);
  int n_final_lists = pl.n_partitions;

  if (pl.path != IC_PATH_UMMA) profile_mark(c, c->ev_score, c->n_ev_score);
  if (pl.path == IC_PATH_GENERIC) {
    for (int q0 = 0; q0 < nq; q0 += GENERIC_QB) {
      e = icc::launch_generic(c->slab, c->size, c->dim, static_cast<const float*>(c->q_f32.p), q0, nq, k,
                              partials, pl.n_partitions, pl.smem_bytes, c->d_status, c->stream);
      if (e != cudaSuccess) return fail(IC_ERR_CUDA, "generic scoring launch failed: %s", cudaGetErrorString(e));
      c->launches += 1;
    }
  } else if (pl.path == IC_PATH_SCAN) {
    for (int q0 = 0; q0 < nq; q0 += pl.query_tile) {
      icc::ScanParams sp;
      sp.slab = c->slab;
      sp.n = c->size;
      sp.dim = c->dim;
      sp.q_f32 = static_cast<const float*>(c->q_f32.p);
      sp.q0 = q0;
      sp.nq = nq;
      sp.qb = pl.query_tile;
      sp.k = k;
      sp.partials = partials;
      sp.n_part = pl.n_partitions;
      sp.n_stages = pl.n_stages;
      sp.rows_per_stage = SCAN_ROWS_PER_STAGE;
      sp.smem_bytes = pl.smem_bytes;
      sp.dev_status = c->d_status;
      e = icc::launch_scan(sp, c->stream);
      if (e != cudaSuccess) return fail(IC_ERR_CUDA, "scan launch failed: %s", cudaGetErrorString(e));
      c->launches += 1;
    }
  } else {
    rc = run_umma_passes(c, pl, direct ? q : c->q_bf16.p, nq, direct ? nq : nq_pad, k, partials,
                         static_cast<uint64_t*>(c->thr.p),
                         static_cast<float*>(c->maxima.p), static_cast<unsigned long long*>(c->pace.p), &n_final_lists,
                         true);
    if (rc != IC_OK) return rc;
  }
  if (pl.path != IC_PATH_UMMA) profile_mark(c, c->ev_score, c->n_ev_score);
  profile_mark(c, c->ev_merge, c->n_ev_merge);
  e = icc::launch_merge(partials, n_final_lists, nq, k, c->ids, out_ids, out_scores, min_score, out_counts, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "merge launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  profile_mark(c, c->ev_merge, c->n_ev_merge);
  return IC_OK;
}

// ------------------------------------------------------------------ allocation-free query
// Scratch of ic_cache_query_static: one fixed array in the library image, per GPU.  In host
// code the symbol below is only a handle for the runtime, not a device address; the address
// is looked up once per device with cudaGetSymbolAddress and cached here.
static __device__ __align__(256) unsigned char g_static_scratch[IC_STATIC_SCRATCH_BYTES];
constexpr int STATIC_MAX_DEVICES = 64;
unsigned char* g_static_scratch_addr[STATIC_MAX_DEVICES] = {};
std::mutex g_static_scratch_mutex;

// Device address of the static scratch on `dev`, which must be the current device.
int static_scratch_address(int dev, unsigned char** out) {
  if (dev < 0 || dev >= STATIC_MAX_DEVICES) return fail(IC_ERR_UNSUPPORTED, "static scratch: device %d out of range", dev);
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (!g_static_scratch_addr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      cudaGetLastError();
      return fail(IC_ERR_CUDA, "cudaGetSymbolAddress of the static scratch failed on device %d: %s", dev, cudaGetErrorString(e));
    }
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_static_scratch_addr[dev];
  return IC_OK;
}

// Where the pieces of a query window's scratch sit inside one fixed block (the static array or a
// caller's workspace), and how much of it the window needs.
struct FixedLayout {
  size_t off_qbf16, off_qf32, off_part, off_thr, off_max, off_pace, need;
};

FixedLayout fixed_layout(int dim, int nq, int k, const ic_cache_plan_t& pl) {
  const int nq_pad = (nq + QUERY_TILE - 1) / QUERY_TILE * QUERY_TILE;
  const size_t list_block = (size_t)nq * k;
  auto round_up = [](size_t v) { return (v + 1023) & ~(size_t)1023; };
  FixedLayout f;
  f.off_pace = 0;   // at a fixed place, whatever the shape
  f.off_qbf16 = PACE_BYTES;
  f.off_qf32 = f.off_qbf16 + round_up((size_t)nq_pad * dim * 2);
  f.off_part = f.off_qf32 + round_up((size_t)nq * dim * 4);
  f.off_thr = f.off_part + round_up((size_t)(2 * pl.n_partitions + 2) * list_block * 8);
  f.off_max = f.off_thr + round_up((size_t)nq * 8);
  f.need = f.off_max + round_up(seed_maxima_bytes(pl));
  return f;
}

// One query window with all scratch taken from a fixed block of `block_bytes` at `base` (NULL: the
// static array of this device).  Mirrors do_query_window but never grows a buffer, creates an
// event or allocates in any other way.
int do_query_window_fixed(ic_cache* c, unsigned char* base, size_t block_bytes, const char* block_name, const void* q,
                          int nq, int k, int64_t* out_ids, float* out_scores, float min_score, int32_t* out_counts) {
  ic_cache_plan_t pl;
  int rc = plan_impl(c->dim, c->size, nq, k, c->forced_path, c->sm_count, c->smem_optin, &pl);
  if (rc != IC_OK) return rc;
  const int nq_pad = (nq + QUERY_TILE - 1) / QUERY_TILE * QUERY_TILE;
  const FixedLayout f = fixed_layout(c->dim, nq, k, pl);
  if (f.need > block_bytes)
    return fail(IC_ERR_NOMEM, "query needs %zu bytes of scratch but the %s holds %zu; use a smaller nq/k or a handle without it",
                f.need, block_name, block_bytes);
  if (!base && (rc = static_scratch_address(c->device, &base)) != IC_OK) return rc;
  void* q_bf16 = base + f.off_qbf16;
  float* q_f32 = reinterpret_cast<float*>(base + f.off_qf32);
  uint64_t* partials = reinterpret_cast<uint64_t*>(base + f.off_part);
  uint64_t* thr = reinterpret_cast<uint64_t*>(base + f.off_thr);
  float* maxima = reinterpret_cast<float*>(base + f.off_max);
  unsigned long long* pace = reinterpret_cast<unsigned long long*>(base + f.off_pace);

  cudaError_t e = icc::launch_convert_rows(q, c->input_dtype == IC_F32, nq, c->dim, c->normalize, q_bf16, q_f32, nq_pad,
                                           nullptr, nullptr, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "query preparation launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  int n_final_lists = pl.n_partitions;
  if (pl.path == IC_PATH_GENERIC) {
    for (int q0 = 0; q0 < nq; q0 += GENERIC_QB) {
      e = icc::launch_generic(c->slab, c->size, c->dim, q_f32, q0, nq, k, partials, pl.n_partitions, pl.smem_bytes,
                              c->d_status, c->stream);
      if (e != cudaSuccess) return fail(IC_ERR_CUDA, "generic scoring launch failed: %s", cudaGetErrorString(e));
      c->launches += 1;
    }
  } else if (pl.path == IC_PATH_SCAN) {
    for (int q0 = 0; q0 < nq; q0 += pl.query_tile) {
      icc::ScanParams sp;
      sp.slab = c->slab;
      sp.n = c->size;
      sp.dim = c->dim;
      sp.q_f32 = q_f32;
      sp.q0 = q0;
      sp.nq = nq;
      sp.qb = pl.query_tile;
      sp.k = k;
      sp.partials = partials;
      sp.n_part = pl.n_partitions;
      sp.n_stages = pl.n_stages;
      sp.rows_per_stage = SCAN_ROWS_PER_STAGE;
      sp.smem_bytes = pl.smem_bytes;
      sp.dev_status = c->d_status;
      e = icc::launch_scan(sp, c->stream);
      if (e != cudaSuccess) return fail(IC_ERR_CUDA, "scan launch failed: %s", cudaGetErrorString(e));
      c->launches += 1;
    }
  } else {
    rc = run_umma_passes(c, pl, q_bf16, nq, nq_pad, k, partials, thr, maxima, pace, &n_final_lists, false);
    if (rc != IC_OK) return rc;
  }
  e = icc::launch_merge(partials, n_final_lists, nq, k, c->ids, out_ids, out_scores, min_score, out_counts, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "merge launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  return IC_OK;
}

// Top-k of `count` stored bf16 rows (q_rows: device, [count, dim]; `readable` rows from q_rows on
// may be read) against the entries of cache c on the tensor-core path, in windows of 1024 rows.
// The query tensor map points straight at the rows: no conversion pass.  self_first < 0:
// out_ids/out_scores are [count, k].  self_first >= 0: the rows are c's own entries from slot
// self_first on and one result per row is written, its best entry other than itself.
int query_bf16_rows(ic_cache* c, const char* q_rows, int64_t count, int64_t readable, int k, int64_t* out_ids,
                    float* out_scores, int64_t self_first) {
  int rc;
  for (int64_t w0 = 0; w0 < count; w0 += WINDOW_MAX_NQ) {
    const int nq = (int)std::min<int64_t>(WINDOW_MAX_NQ, count - w0);
    ic_cache_plan_t pl;
    if ((rc = plan_impl(c->dim, c->size, nq, k, IC_PATH_UMMA, c->sm_count, c->smem_optin, &pl)) != IC_OK) return rc;
    const size_t list_block = (size_t)nq * k;
    if ((rc = ensure(c, c->partials, (size_t)(2 * pl.n_partitions + 2) * list_block * 8, "partial top-k lists")) != IC_OK) return rc;
    if ((rc = ensure(c, c->thr, (size_t)nq * 8, "seed thresholds")) != IC_OK) return rc;
    if ((rc = ensure(c, c->maxima, seed_maxima_bytes(pl), "group maxima")) != IC_OK) return rc;
    uint64_t* partials = static_cast<uint64_t*>(c->partials.p);
    int n_final_lists = 0;
    // the map may cover following rows up to a full 128-row tile, never past `readable`; lanes
    // beyond nq are not real queries, whatever they read
    const int q_map_rows = (int)std::min<int64_t>((nq + QUERY_TILE - 1) / QUERY_TILE * QUERY_TILE, readable - w0);
    rc = run_umma_passes(c, pl, q_rows + (size_t)w0 * c->dim * 2, nq, q_map_rows, k, partials,
                         static_cast<uint64_t*>(c->thr.p), static_cast<float*>(c->maxima.p),
                         static_cast<unsigned long long*>(c->pace.p), &n_final_lists, false);
    if (rc != IC_OK) return rc;
    const size_t out_stride = self_first >= 0 ? 1 : (size_t)k;
    cudaError_t e = icc::launch_merge(partials, n_final_lists, nq, k, c->ids, out_ids + (size_t)w0 * out_stride,
                                      out_scores + (size_t)w0 * out_stride, -INFINITY, nullptr, c->stream,
                                      self_first >= 0 ? self_first + w0 : -1);
    if (e != cudaSuccess) return fail(IC_ERR_CUDA, "merge launch failed: %s", cudaGetErrorString(e));
    c->launches += 1;
  }
  return IC_OK;
}

void drop_index(ic_cache* c) {
  if (c->centroids) {
    ic_cache_destroy(c->centroids);
    c->centroids = nullptr;
  }
  c->n_clusters = 0;
  c->n_indexed = 0;
  c->have_idx_rows = false;
}

int check_query_args(ic_cache* c, const void* q, int32_t nq, int32_t k, const void* out_ids, const void* out_scores) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (nq < 0) return fail(IC_ERR_INVALID, "nq %d < 0", nq);
  if (k < 1 || k > IC_MAX_K) return fail(IC_ERR_INVALID, "k %d outside [1, %d]", k, IC_MAX_K);
  if (nq > 0 && (!q || !out_ids || !out_scores)) return fail(IC_ERR_INVALID, "NULL pointer with nq > 0");
  return IC_OK;
}

}  // namespace

extern "C" {

const char* ic_cache_last_error(void) { return g_err; }

int32_t ic_cache_version(void) { return 100; }

int ic_cache_plan(int32_t dim, int64_t n, int32_t nq, int32_t k, int32_t path, int32_t sm_count,
                  int32_t smem_optin, ic_cache_plan_t* plan) {
  return plan_impl(dim, n, nq, k, path, sm_count, smem_optin, plan);
}

ic_cache_t* ic_cache_create(int32_t dim, int64_t capacity) { return ic_cache_create_ex(dim, capacity, nullptr); }

ic_cache_t* ic_cache_create_ex(int32_t dim, int64_t capacity, const ic_cache_opts_t* opts) {
  g_err[0] = 0;
  if (dim < 8 || dim > IC_MAX_DIM || (dim % 8) != 0) {
    fail(IC_ERR_INVALID, "dim %d must be a multiple of 8 in [8, %d]", dim, IC_MAX_DIM);
    return nullptr;
  }
  if (capacity < 1 || capacity > 0x7fffffffll - 511) {
    fail(IC_ERR_INVALID, "capacity %lld outside [1, 2^31-512]", (long long)capacity);
    return nullptr;
  }
  ic_cache_opts_t o;
  memset(&o, 0, sizeof o);
  o.device = -1;
  if (opts) {
    if (opts->struct_size < sizeof(uint32_t) || opts->struct_size > sizeof o) {
      fail(IC_ERR_INVALID, "opts.struct_size %u not understood (this build: %zu)", opts->struct_size, sizeof o);
      return nullptr;
    }
    memcpy(&o, opts, opts->struct_size);
  }
  if (o.input_dtype != IC_BF16 && o.input_dtype != IC_F32) {
    fail(IC_ERR_INVALID, "unknown input_dtype %d", o.input_dtype);
    return nullptr;
  }
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    fail(IC_ERR_CUDA, "no usable CUDA device (%s); this library has no CPU fallback",
         e != cudaSuccess ? cudaGetErrorString(e) : "device count is 0");
    return nullptr;
  }
  int dev = o.device;
  if (dev < 0 && cudaGetDevice(&dev) != cudaSuccess) {
    fail(IC_ERR_CUDA, "cudaGetDevice failed");
    return nullptr;
  }
  if (dev >= ndev) {
    fail(IC_ERR_INVALID, "device %d does not exist (%d devices)", dev, ndev);
    return nullptr;
  }
  DeviceGuard guard(dev);
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    fail(IC_ERR_CUDA, "cudaGetDeviceProperties failed");
    return nullptr;
  }
  if (prop.major != 10) {
    fail(IC_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only", dev, prop.major, prop.minor);
    return nullptr;
  }
  ic_cache* c = new (std::nothrow) ic_cache();
  if (!c) {
    fail(IC_ERR_NOMEM, "host allocation failed");
    return nullptr;
  }
  c->device = dev;
  c->dim = dim;
  c->capacity = capacity;
  c->input_dtype = o.input_dtype;
  c->normalize = o.normalize ? 1 : 0;
  c->stream = static_cast<cudaStream_t>(o.stream);
  c->workspace = static_cast<unsigned char*>(o.workspace);
  c->workspace_bytes = o.workspace ? o.workspace_bytes : 0;
  c->sm_count = prop.multiProcessorCount;
  c->smem_optin = (int)prop.sharedMemPerBlockOptin;
  c->l2_bytes = prop.l2CacheSize;

  bool ok = true;
  if (o.slab) {
    if (!is_device_ptr(o.slab, dev) || (reinterpret_cast<uintptr_t>(o.slab) & 255)) {
      fail(IC_ERR_INVALID, "opts.slab must be a 256-byte aligned device pointer on device %d", dev);
      ok = false;
    }
    c->slab = o.slab;
  } else {
    e = cudaMalloc(&c->slab, (size_t)capacity * dim * 2);
    if (e != cudaSuccess) {
      cudaGetLastError();
      fail(IC_ERR_NOMEM, "cudaMalloc of the %zu-byte slab failed: %s", (size_t)capacity * dim * 2, cudaGetErrorString(e));
      c->slab = nullptr;
      ok = false;
    }
    c->own_slab = ok;
  }
  if (ok && o.workspace) {
    if (!is_device_ptr(o.workspace, dev) || (reinterpret_cast<uintptr_t>(o.workspace) & 255)) {
      fail(IC_ERR_INVALID, "opts.workspace must be a 256-byte aligned device pointer on device %d", dev);
      ok = false;
    } else if (c->workspace_bytes >= PACE_BYTES && cudaMemset(o.workspace, 0, PACE_BYTES) != cudaSuccess) {
      // the words the CTAs of a launch exchange start out cleared
      cudaGetLastError();
      fail(IC_ERR_CUDA, "clearing the head of opts.workspace failed");
      ok = false;
    }
  }
  if (ok) {
    if (o.ids) {
      if (!is_device_ptr(o.ids, dev)) {
        fail(IC_ERR_INVALID, "opts.ids must be a device pointer on device %d", dev);
        ok = false;
      }
      c->ids = static_cast<int64_t*>(o.ids);
    } else {
      e = cudaMalloc(reinterpret_cast<void**>(&c->ids), (size_t)capacity * 8);
      if (e != cudaSuccess) {
        cudaGetLastError();
        fail(IC_ERR_NOMEM, "cudaMalloc of the id array failed: %s", cudaGetErrorString(e));
        c->ids = nullptr;
        ok = false;
      }
      c->own_ids = ok;
    }
  }
  if (ok) {
    e = cudaHostAlloc(reinterpret_cast<void**>(&c->h_status), sizeof(int), cudaHostAllocMapped);
    if (e == cudaSuccess) {
      *c->h_status = 0;
      e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->d_status), c->h_status, 0);
    }
    if (e != cudaSuccess) {
      cudaGetLastError();
      fail(IC_ERR_CUDA, "status word allocation failed: %s", cudaGetErrorString(e));
      ok = false;
    }
  }
  if (ok) {
    e = cudaMalloc(&c->pace.p, PACE_BYTES);
    if (e == cudaSuccess) e = cudaMemset(c->pace.p, 0, PACE_BYTES);
    if (e != cudaSuccess) {
      cudaGetLastError();
      fail(IC_ERR_NOMEM, "cudaMalloc of the pacing words failed: %s", cudaGetErrorString(e));
      c->pace.p = nullptr;
      ok = false;
    } else {
      c->pace.bytes = PACE_BYTES;
    }
  }
  if (ok) {
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
      cudaGetLastError();
      fail(IC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
      ok = false;
    } else {
      c->encode = reinterpret_cast<EncodeTiledFn>(fn);
      ok = encode_2d(c, &c->tmap_slab, c->slab, (uint64_t)capacity, ROW_TILE) == IC_OK &&
           encode_2d(c, &c->tmap_slab_half, c->slab, (uint64_t)capacity, ROW_TILE / 2) == IC_OK;
      c->have_tmap_slab = ok;
    }
  }
  if (ok) {
    cudaError_t e1 = icc::merge_configure(c->smem_optin);
    cudaError_t e2 = icc::scan_configure(c->smem_optin);
    cudaError_t e3 = icc::umma_configure(c->smem_optin);
    if (e3 == cudaSuccess) e3 = icc::index_configure(c->smem_optin);
    if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) {
      cudaGetLastError();
      fail(IC_ERR_CUDA, "kernel attribute set-up failed (merge %d, scan %d, tensor-core %d)", (int)e1, (int)e2, (int)e3);
      ok = false;
    }
  }
  if (!ok) {
    char keep[sizeof g_err];
    memcpy(keep, g_err, sizeof keep);
    ic_cache_destroy(c);
    memcpy(g_err, keep, sizeof keep);
    return nullptr;
  }
  return c;
}

void ic_cache_destroy(ic_cache_t* c) {
  if (!c) return;
  DeviceGuard guard(c->device);
  cudaStreamSynchronize(c->stream);
  drop_index(c);
  if (c->utility) cudaFree(c->utility);
  release(c->util_ids);
  release(c->util_gains);
  release(c->idx_assign);
  release(c->idx_best);
  release(c->idx_order);
  release(c->idx_offsets);
  release(c->idx_sort);
  release(c->idx_init);
  release(c->idx_probes);
  release(c->idx_probe_scores);
  release(c->idx_rows);
  if (c->own_slab && c->slab) cudaFree(c->slab);
  if (c->own_ids && c->ids) cudaFree(c->ids);
  release(c->q_bf16);
  release(c->q_f32);
  release(c->partials);
  release(c->thr);
  release(c->maxima);
  release(c->pace);
  release(c->stage_in);
  release(c->stage_ids);
  release(c->stage_scores);
  release(c->evict);
  if (c->h_status) cudaFreeHost(c->h_status);
  for (cudaEvent_t ev : c->ev_score) cudaEventDestroy(ev);
  for (cudaEvent_t ev : c->ev_merge) cudaEventDestroy(ev);
  for (cudaEvent_t ev : c->ev_seed) cudaEventDestroy(ev);
  cudaGetLastError();
  delete c;
}

int ic_cache_insert(ic_cache_t* c, const void* emb, const int64_t* ids, int64_t n) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (n < 0) return fail(IC_ERR_INVALID, "n %lld < 0", (long long)n);
  if (n == 0) return IC_OK;
  if (!emb || !ids) return fail(IC_ERR_INVALID, "NULL pointer with n > 0");
  if (c->size + n > c->capacity)
    return fail(IC_ERR_FULL, "insert of %lld rows exceeds capacity (%lld of %lld used)", (long long)n, (long long)c->size, (long long)c->capacity);
  DeviceGuard guard(c->device);
  if (!is_device_ptr(emb, c->device) || !is_device_ptr(ids, c->device))
    return fail(IC_ERR_INVALID, "emb and ids must be device pointers on device %d (use ic_cache_insert_host for host memory)", c->device);
  int rc = check_timeout(c);
  if (rc != IC_OK) return rc;
  return do_insert(c, emb, ids, n);
}

int ic_cache_insert_host(ic_cache_t* c, const void* emb_host, const int64_t* ids_host, int64_t n) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (n < 0) return fail(IC_ERR_INVALID, "n %lld < 0", (long long)n);
  if (n == 0) return IC_OK;
  if (!emb_host || !ids_host) return fail(IC_ERR_INVALID, "NULL pointer with n > 0");
  if (c->size + n > c->capacity)
    return fail(IC_ERR_FULL, "insert of %lld rows exceeds capacity (%lld of %lld used)", (long long)n, (long long)c->size, (long long)c->capacity);
  DeviceGuard guard(c->device);
  int rc = check_timeout(c);
  if (rc != IC_OK) return rc;
  // stage in slices so that a large bulk load needs only a bounded device buffer
  const int64_t slice = std::max<int64_t>(1, (int64_t)(64u << 20) / ((int64_t)c->dim * (int64_t)in_elem_bytes(c)));
  const size_t row_bytes = (size_t)c->dim * in_elem_bytes(c);
  if ((rc = ensure(c, c->stage_in, (size_t)std::min(slice, n) * row_bytes, "insert staging")) != IC_OK) return rc;
  if ((rc = ensure(c, c->stage_ids, (size_t)std::min(slice, n) * 8, "insert id staging")) != IC_OK) return rc;
  const int64_t size_before = c->size;
  for (int64_t r0 = 0; r0 < n; r0 += slice) {
    const int64_t rows = std::min(slice, n - r0);
    cudaError_t e = cudaMemcpyAsync(c->stage_in.p, static_cast<const char*>(emb_host) + (size_t)r0 * row_bytes,
                                    (size_t)rows * row_bytes, cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(c->stage_ids.p, ids_host + r0, (size_t)rows * 8, cudaMemcpyHostToDevice, c->stream);
    if (e != cudaSuccess) {
      c->size = size_before;
      return fail(IC_ERR_CUDA, "host-to-device copy failed: %s", cudaGetErrorString(e));
    }
    rc = do_insert(c, c->stage_in.p, static_cast<const int64_t*>(c->stage_ids.p), rows);
    if (rc != IC_OK) {
      c->size = size_before;
      return rc;
    }
    if (r0 + slice < n && cudaStreamSynchronize(c->stream) != cudaSuccess) {  // staging is reused
      c->size = size_before;
      return fail(IC_ERR_CUDA, "stream sync failed during host insert");
    }
  }
  // No final synchronisation: the device staging buffer is only reused by work enqueued later
  // on the same stream, and pageable host memory has been copied out by the time
  // cudaMemcpyAsync returns; pinned host buffers must stay untouched until a synchronising call.
  return IC_OK;
}

int ic_cache_query(ic_cache_t* c, const void* q, int32_t nq, int32_t k, int64_t* out_ids, float* out_scores) {
  return ic_cache_query_min_score(c, q, nq, k, -INFINITY, out_ids, out_scores, nullptr);
}

int ic_cache_query_min_score(ic_cache_t* c, const void* q, int32_t nq, int32_t k, float min_score, int64_t* out_ids,
                             float* out_scores, int32_t* out_counts) {
  int rc = check_query_args(c, q, nq, k, out_ids, out_scores);
  if (rc != IC_OK || nq == 0) return rc;
  if (min_score != min_score) return fail(IC_ERR_INVALID, "min_score is NaN");
  DeviceGuard guard(c->device);
  if (out_counts && !is_device_ptr(out_counts, c->device))
    return fail(IC_ERR_INVALID, "out_counts must be a device pointer on device %d", c->device);
  if (!is_device_ptr(q, c->device) || !is_device_ptr(out_ids, c->device) || !is_device_ptr(out_scores, c->device))
    return fail(IC_ERR_INVALID, "q, out_ids and out_scores must be device pointers on device %d (use ic_cache_query_host for host memory)", c->device);
  if ((rc = check_timeout(c)) != IC_OK) return rc;
  const size_t q_row = (size_t)c->dim * in_elem_bytes(c);
  for (int q0 = 0; q0 < nq; q0 += WINDOW_MAX_NQ) {
    const int w = std::min(WINDOW_MAX_NQ, nq - q0);
    const char* qw = static_cast<const char*>(q) + (size_t)q0 * q_row;
    if (c->workspace)   // caller-owned scratch: nothing is allocated, too small a workspace is an error
      rc = do_query_window_fixed(c, c->workspace, c->workspace_bytes, "caller's workspace", qw, w, k,
                                 out_ids + (size_t)q0 * k, out_scores + (size_t)q0 * k, min_score,
                                 out_counts ? out_counts + q0 : nullptr);
    else
      rc = do_query_window(c, qw, w, k, out_ids + (size_t)q0 * k, out_scores + (size_t)q0 * k, min_score,
                           out_counts ? out_counts + q0 : nullptr);
    if (rc != IC_OK) return rc;
  }
  return IC_OK;
}

size_t ic_cache_workspace_bytes(int32_t dim, int64_t capacity, int32_t max_nq, int32_t max_k) {
  if (dim < 8 || dim > IC_MAX_DIM || (dim % 8) != 0 || capacity < 1 || max_nq < 1 || max_k < 1 || max_k > IC_MAX_K) {
    fail(IC_ERR_INVALID, "workspace_bytes: bad dim, capacity, max_nq or max_k");
    return 0;
  }
  // the launch plan depends on the device: the current one when there is one, else a B200's figures
  int sm_count = 148, smem_optin = 232448, dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaGetDeviceProperties(&prop, dev) == cudaSuccess) {
    sm_count = prop.multiProcessorCount;
    smem_optin = (int)prop.sharedMemPerBlockOptin;
  } else {
    cudaGetLastError();
  }
  // a call is served in windows of at most 1024 queries; within a given number of query tiles the
  // need grows with nq, so the largest batch of every tile count (and one or two queries, which
  // may take the scan path) covers all shapes
  const int limit = std::min<int>(max_nq, WINDOW_MAX_NQ);
  size_t need = 0;
  for (int cand = 0; cand <= WINDOW_MAX_NQ / QUERY_TILE + 1; ++cand) {
    const int nq = cand == 0 ? 1 : (cand == 1 ? std::min(2, limit) : std::min((cand - 1) * QUERY_TILE, limit));
    for (int path : {(int)IC_PATH_AUTO, (int)IC_PATH_UMMA}) {
      ic_cache_plan_t pl;
      if (plan_impl(dim, capacity, nq, max_k, path, sm_count, smem_optin, &pl) != IC_OK) continue;
      need = std::max(need, fixed_layout(dim, nq, max_k, pl).need);
    }
  }
  return need;
}

int ic_cache_query_static(ic_cache_t* c, const void* q, int32_t nq, int32_t k, int64_t* out_ids, float* out_scores) {
  int rc = check_query_args(c, q, nq, k, out_ids, out_scores);
  if (rc != IC_OK || nq == 0) return rc;
  if (nq > WINDOW_MAX_NQ) return fail(IC_ERR_INVALID, "ic_cache_query_static takes at most %d queries per call", WINDOW_MAX_NQ);
  DeviceGuard guard(c->device);
  if (!is_device_ptr(q, c->device) || !is_device_ptr(out_ids, c->device) || !is_device_ptr(out_scores, c->device))
    return fail(IC_ERR_INVALID, "q, out_ids and out_scores must be device pointers on device %d", c->device);
  if ((rc = check_timeout(c)) != IC_OK) return rc;
  return do_query_window_fixed(c, nullptr, IC_STATIC_SCRATCH_BYTES, "static scratch", q, nq, k, out_ids, out_scores,
                               -INFINITY, nullptr);
}

int ic_cache_query_host(ic_cache_t* c, const void* q_host, int32_t nq, int32_t k, int64_t* out_ids_host,
                        float* out_scores_host) {
  int rc = check_query_args(c, q_host, nq, k, out_ids_host, out_scores_host);
  if (rc != IC_OK || nq == 0) return rc;
  DeviceGuard guard(c->device);
  if ((rc = check_timeout(c)) != IC_OK) return rc;
  const size_t q_bytes = (size_t)nq * c->dim * in_elem_bytes(c);
  if ((rc = ensure(c, c->stage_in, q_bytes, "query input staging")) != IC_OK) return rc;
  if ((rc = ensure(c, c->stage_ids, (size_t)nq * k * 8, "result id staging")) != IC_OK) return rc;
  if ((rc = ensure(c, c->stage_scores, (size_t)nq * k * 4, "result score staging")) != IC_OK) return rc;
  cudaError_t e = cudaMemcpyAsync(c->stage_in.p, q_host, q_bytes, cudaMemcpyHostToDevice, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "host-to-device copy failed: %s", cudaGetErrorString(e));
  const size_t q_row = (size_t)c->dim * in_elem_bytes(c);
  for (int q0 = 0; q0 < nq; q0 += WINDOW_MAX_NQ) {
    const int w = std::min(WINDOW_MAX_NQ, nq - q0);
    rc = do_query_window(c, static_cast<const char*>(c->stage_in.p) + (size_t)q0 * q_row, w, k,
                         static_cast<int64_t*>(c->stage_ids.p) + (size_t)q0 * k,
                         static_cast<float*>(c->stage_scores.p) + (size_t)q0 * k, -INFINITY, nullptr);
    if (rc != IC_OK) return rc;
  }
  e = cudaMemcpyAsync(out_ids_host, c->stage_ids.p, (size_t)nq * k * 8, cudaMemcpyDeviceToHost, c->stream);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(out_scores_host, c->stage_scores.p, (size_t)nq * k * 4, cudaMemcpyDeviceToHost, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "result copy failed: %s", cudaGetErrorString(e));
  return check_timeout(c);
}

int ic_cache_remove(ic_cache_t* c, const int64_t* ids_host, int64_t n, int64_t* n_removed) {
  if (n_removed) *n_removed = 0;
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (n < 0) return fail(IC_ERR_INVALID, "n %lld < 0", (long long)n);
  if (n == 0 || c->size == 0) return IC_OK;
  if (!ids_host) return fail(IC_ERR_INVALID, "NULL pointer with n > 0");
  DeviceGuard guard(c->device);
  int rc = check_timeout(c);
  if (rc != IC_OK) return rc;
  // the ids to drop, sorted and without repeats
  std::vector<int64_t> wanted(ids_host, ids_host + n);
  std::sort(wanted.begin(), wanted.end());
  wanted.erase(std::unique(wanted.begin(), wanted.end()), wanted.end());
  const int64_t nw = (int64_t)wanted.size();
  // device scratch: [wanted nw][count 1][matches cap][src cap][dst cap]
  const int64_t cap = std::min<int64_t>(c->size, 4 * nw + 1024);
  const size_t words = (size_t)nw + 1 + 3 * (size_t)cap;
  if ((rc = ensure(c, c->evict, words * 8, "eviction scratch")) != IC_OK) return rc;
  int64_t* d_wanted = static_cast<int64_t*>(c->evict.p);
  unsigned long long* d_count = reinterpret_cast<unsigned long long*>(d_wanted + nw);
  int64_t* d_match = d_wanted + nw + 1;
  int64_t* d_src = d_match + cap;
  int64_t* d_dst = d_src + cap;
  cudaError_t e = cudaMemcpyAsync(d_wanted, wanted.data(), (size_t)nw * 8, cudaMemcpyHostToDevice, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(d_count, 0, 8, c->stream);
  if (e == cudaSuccess) e = icc::launch_find_ids(c->ids, c->size, d_wanted, nw, d_match, d_count, cap, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "id search launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  unsigned long long m = 0;
  e = cudaMemcpyAsync(&m, d_count, 8, cudaMemcpyDeviceToHost, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "id search failed: %s", cudaGetErrorString(e));
  if (m == 0) return IC_OK;
  if ((int64_t)m > cap)
    return fail(IC_ERR_UNSUPPORTED, "%llu entries carry the %lld given ids (more than %lld): remove them in smaller groups",
                m, (long long)nw, (long long)cap);
  std::vector<int64_t> gone((size_t)m);
  e = cudaMemcpy(gone.data(), d_match, (size_t)m * 8, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "match copy failed: %s", cudaGetErrorString(e));
  std::sort(gone.begin(), gone.end());
  // vacated slots below the new size are refilled, in order, by the surviving rows of the tail
  const int64_t new_size = c->size - (int64_t)m;
  std::vector<int64_t> src, dst;
  size_t gi = std::lower_bound(gone.begin(), gone.end(), new_size) - gone.begin();   // first removed slot in the tail
  int64_t tail = new_size;
  for (size_t h = 0; h < gone.size() && gone[h] < new_size; ++h) {
    while (gi < gone.size() && gone[gi] == tail) {   // skip tail rows that are removed themselves
      ++gi;
      ++tail;
    }
    dst.push_back(gone[h]);
    src.push_back(tail++);
  }
  if (!src.empty()) {
    e = cudaMemcpyAsync(d_src, src.data(), src.size() * 8, cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_dst, dst.data(), dst.size() * 8, cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess) e = icc::launch_move_rows(c->slab, c->ids, c->utility, d_src, d_dst, (int64_t)src.size(), c->dim, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // src/dst are host vectors about to go away
    if (e != cudaSuccess) return fail(IC_ERR_CUDA, "row move failed: %s", cudaGetErrorString(e));
    c->launches += 1;
  }
  c->size = new_size;
  if (n_removed) *n_removed = (int64_t)m;
  drop_index(c);   // rows moved: member lists and assignments no longer name the right slots
  return IC_OK;
}

int ic_cache_self_similarity(ic_cache_t* c, int64_t first, int64_t count, int64_t* out_ids, float* out_scores) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (first < 0 || count < 0 || first + count > c->size)
    return fail(IC_ERR_INVALID, "rows [%lld, %lld) are not all cached (size %lld)", (long long)first, (long long)(first + count), (long long)c->size);
  if (count == 0) return IC_OK;
  if (!out_ids || !out_scores) return fail(IC_ERR_INVALID, "NULL pointer with count > 0");
  DeviceGuard guard(c->device);
  if (!is_device_ptr(out_ids, c->device) || !is_device_ptr(out_scores, c->device))
    return fail(IC_ERR_INVALID, "out_ids and out_scores must be device pointers on device %d", c->device);
  int rc = check_timeout(c);
  if (rc != IC_OK) return rc;
  const int k = 2;   // a row's best match is itself or an exact copy; the next one is the answer
  const char* q_rows = static_cast<const char*>(c->slab) + (size_t)first * c->dim * 2;
  return query_bf16_rows(c, q_rows, count, c->capacity - first, k, out_ids, out_scores, first);
}

// ------------------------------------------------------------------ checkpoint file
// Layout: a 64-byte header, then size*dim bf16 rows, size int64 ids, and (flag) size fp32 utilities.
namespace {
struct CheckpointHeader {
  char magic[8];        // "ICCKPT01"
  int32_t dim;
  int32_t has_utility;
  int64_t size;
  int64_t reserved[5];
};
static_assert(sizeof(CheckpointHeader) == 64, "checkpoint header is 64 bytes");
constexpr size_t CKPT_CHUNK = (size_t)32 << 20;

// Stream `bytes` between a device range and the file through a host bounce buffer.
int copy_device_file(void* dev, size_t bytes, FILE* f, bool to_file, std::vector<unsigned char>& bounce, const char* path) {
  for (size_t off = 0; off < bytes; off += CKPT_CHUNK) {
    const size_t len = std::min(CKPT_CHUNK, bytes - off);
    if (to_file) {
      if (cudaMemcpy(bounce.data(), static_cast<char*>(dev) + off, len, cudaMemcpyDeviceToHost) != cudaSuccess)
        return fail(IC_ERR_CUDA, "device-to-host copy failed while writing %s", path);
      if (fwrite(bounce.data(), 1, len, f) != len) return fail(IC_ERR_INVALID, "short write to %s", path);
    } else {
      if (fread(bounce.data(), 1, len, f) != len) return fail(IC_ERR_INVALID, "%s is truncated", path);
      if (cudaMemcpy(static_cast<char*>(dev) + off, bounce.data(), len, cudaMemcpyHostToDevice) != cudaSuccess)
        return fail(IC_ERR_CUDA, "host-to-device copy failed while reading %s", path);
    }
  }
  return IC_OK;
}
}  // namespace

int ic_cache_save(ic_cache_t* c, const char* path) {
  if (!c || !path) return fail(IC_ERR_INVALID, "NULL handle or path");
  DeviceGuard guard(c->device);
  int rc = ic_cache_sync(c);
  if (rc != IC_OK) return rc;
  FILE* f = fopen(path, "wb");
  if (!f) return fail(IC_ERR_INVALID, "cannot open %s for writing", path);
  CheckpointHeader h;
  memset(&h, 0, sizeof h);
  memcpy(h.magic, "ICCKPT01", 8);
  h.dim = c->dim;
  h.has_utility = c->utility ? 1 : 0;
  h.size = c->size;
  std::vector<unsigned char> bounce(std::min(CKPT_CHUNK, std::max<size_t>(1, (size_t)c->size * c->dim * 2)));
  rc = fwrite(&h, sizeof h, 1, f) == 1 ? IC_OK : fail(IC_ERR_INVALID, "short write to %s", path);
  if (rc == IC_OK) rc = copy_device_file(c->slab, (size_t)c->size * c->dim * 2, f, true, bounce, path);
  if (rc == IC_OK) rc = copy_device_file(c->ids, (size_t)c->size * 8, f, true, bounce, path);
  if (rc == IC_OK && c->utility) rc = copy_device_file(c->utility, (size_t)c->size * 4, f, true, bounce, path);
  if (fclose(f) != 0 && rc == IC_OK) rc = fail(IC_ERR_INVALID, "closing %s failed", path);
  return rc;
}

int ic_cache_load(ic_cache_t* c, const char* path) {
  if (!c || !path) return fail(IC_ERR_INVALID, "NULL handle or path");
  DeviceGuard guard(c->device);
  int rc = ic_cache_sync(c);
  if (rc != IC_OK) return rc;
  FILE* f = fopen(path, "rb");
  if (!f) return fail(IC_ERR_INVALID, "cannot open %s", path);
  CheckpointHeader h;
  if (fread(&h, sizeof h, 1, f) != 1 || memcmp(h.magic, "ICCKPT01", 8) != 0) {
    fclose(f);
    return fail(IC_ERR_INVALID, "%s is not a cache checkpoint", path);
  }
  if (h.dim != c->dim || h.size < 0 || h.size > c->capacity) {
    fclose(f);
    return fail(IC_ERR_INVALID, "%s holds %lld entries of dimension %d; this handle has dimension %d and capacity %lld",
                path, (long long)h.size, h.dim, c->dim, (long long)c->capacity);
  }
  if (h.has_utility && (rc = ensure_utility(c)) != IC_OK) {
    fclose(f);
    return rc;
  }
  // from here on the old contents are gone, whatever happens
  drop_index(c);
  c->size = 0;
  std::vector<unsigned char> bounce(std::min(CKPT_CHUNK, std::max<size_t>(1, (size_t)h.size * c->dim * 2)));
  rc = copy_device_file(c->slab, (size_t)h.size * c->dim * 2, f, false, bounce, path);
  if (rc == IC_OK) rc = copy_device_file(c->ids, (size_t)h.size * 8, f, false, bounce, path);
  if (rc == IC_OK && h.has_utility) rc = copy_device_file(c->utility, (size_t)h.size * 4, f, false, bounce, path);
  if (rc == IC_OK && !h.has_utility && c->utility && h.size > 0 &&
      cudaMemset(c->utility, 0, (size_t)h.size * 4) != cudaSuccess)
    rc = fail(IC_ERR_CUDA, "clearing the utility array failed");
  fclose(f);
  if (rc == IC_OK) c->size = h.size;
  return rc;
}

int ic_cache_utility_add(ic_cache_t* c, const int64_t* ids_host, const float* gains_host, int64_t n) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (n < 0) return fail(IC_ERR_INVALID, "n %lld < 0", (long long)n);
  if (n == 0) return IC_OK;
  if (!ids_host || !gains_host) return fail(IC_ERR_INVALID, "NULL pointer with n > 0");
  for (int64_t i = 0; i < n; ++i)
    if (!(gains_host[i] == gains_host[i]) || fabsf(gains_host[i]) == INFINITY) return fail(IC_ERR_INVALID, "gain %lld is not finite", (long long)i);
  DeviceGuard guard(c->device);
  int rc = check_timeout(c);
  if (rc != IC_OK) return rc;
  if ((rc = ensure_utility(c)) != IC_OK) return rc;
  // sort by id, keeping the caller's order among equal ids
  std::vector<int64_t> perm((size_t)n);
  for (int64_t i = 0; i < n; ++i) perm[(size_t)i] = i;
  std::stable_sort(perm.begin(), perm.end(), [&](int64_t a, int64_t b) { return ids_host[a] < ids_host[b]; });
  std::vector<int64_t> ids((size_t)n);
  std::vector<float> gains((size_t)n);
  for (int64_t i = 0; i < n; ++i) {
    ids[(size_t)i] = ids_host[perm[(size_t)i]];
    gains[(size_t)i] = gains_host[perm[(size_t)i]];
  }
  if ((rc = ensure(c, c->util_ids, (size_t)n * 8, "utility update ids")) != IC_OK) return rc;
  if ((rc = ensure(c, c->util_gains, (size_t)n * 4, "utility update gains")) != IC_OK) return rc;
  cudaError_t e = cudaMemcpyAsync(c->util_ids.p, ids.data(), (size_t)n * 8, cudaMemcpyHostToDevice, c->stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(c->util_gains.p, gains.data(), (size_t)n * 4, cudaMemcpyHostToDevice, c->stream);
  if (e == cudaSuccess)
    e = icc::launch_utility_add(c->ids, c->size, static_cast<const int64_t*>(c->util_ids.p),
                                static_cast<const float*>(c->util_gains.p), n, c->utility, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // the sorted copies are host vectors about to go away
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "utility update failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  return IC_OK;
}

int ic_cache_utility_decay(ic_cache_t* c, float factor) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (!(factor >= 0.0f) || factor == INFINITY) return fail(IC_ERR_INVALID, "decay factor must be finite and >= 0");
  if (!c->utility || c->size == 0) return IC_OK;   // all utilities are zero
  DeviceGuard guard(c->device);
  int rc = check_timeout(c);
  if (rc != IC_OK) return rc;
  cudaError_t e = icc::launch_utility_scale(c->utility, c->size, factor, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "utility decay launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  return IC_OK;
}

int ic_cache_utility_read(ic_cache_t* c, int64_t* ids_host, float* utility_host) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (c->size == 0) return IC_OK;
  DeviceGuard guard(c->device);
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e == cudaSuccess && ids_host) e = cudaMemcpy(ids_host, c->ids, (size_t)c->size * 8, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && utility_host) {
    if (c->utility) e = cudaMemcpy(utility_host, c->utility, (size_t)c->size * 4, cudaMemcpyDeviceToHost);
    else memset(utility_host, 0, (size_t)c->size * 4);
  }
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "utility copy failed: %s", cudaGetErrorString(e));
  return IC_OK;
}

int ic_cache_build_index(ic_cache_t* c, int32_t n_clusters, int32_t n_iters, const int64_t* init_slots_host) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (c->size < 1) return fail(IC_ERR_INVALID, "cannot cluster an empty cache");
  if (n_iters < 0) return fail(IC_ERR_INVALID, "n_iters %d < 0", n_iters);
  const int64_t k_max = std::min<int64_t>(c->size, IC_MAX_CLUSTERS);
  int64_t K = n_clusters;
  if (n_clusters == 0) K = std::max<int64_t>(1, std::min<int64_t>(k_max, llround(sqrt((double)c->size))));
  if (K < 1 || K > k_max) return fail(IC_ERR_INVALID, "n_clusters %d outside [1, %lld]", n_clusters, (long long)k_max);
  std::vector<int64_t> init((size_t)K);
  if (init_slots_host) {
    std::vector<int64_t> sorted(init_slots_host, init_slots_host + K);
    std::sort(sorted.begin(), sorted.end());
    for (int64_t i = 0; i < K; ++i) {
      if (sorted[i] < 0 || sorted[i] >= c->size || (i > 0 && sorted[i] == sorted[i - 1]))
        return fail(IC_ERR_INVALID, "init_slots must be %lld distinct slots in [0, %lld)", (long long)K, (long long)c->size);
      init[i] = init_slots_host[i];
    }
  } else {
    for (int64_t i = 0; i < K; ++i) init[i] = i * c->size / K;
  }
  DeviceGuard guard(c->device);
  int rc = check_timeout(c);
  if (rc != IC_OK) return rc;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(IC_ERR_CUDA, "stream sync failed");
  drop_index(c);
  const int64_t n = c->size;
  if ((rc = ensure(c, c->idx_init, (size_t)K * 8, "initial centroid slots")) != IC_OK) return rc;
  if ((rc = ensure(c, c->idx_assign, (size_t)n * 8, "cluster assignments")) != IC_OK) return rc;
  if ((rc = ensure(c, c->idx_best, (size_t)n * 4, "assignment scores")) != IC_OK) return rc;
  if ((rc = ensure(c, c->idx_order, (size_t)n * 4, "cluster member lists")) != IC_OK) return rc;
  if ((rc = ensure(c, c->idx_offsets, (size_t)(K + 1) * 4, "cluster offsets")) != IC_OK) return rc;
  if ((rc = ensure(c, c->idx_sort, icc::sort_scratch_ints(n, (int)K) * 4, "sort scratch")) != IC_OK) return rc;
  // the child shares device, stream and input conventions, so a query's centroid step sees the
  // same bf16-rounded query as the scan of the clusters
  ic_cache_opts_t o;
  memset(&o, 0, sizeof o);
  o.struct_size = sizeof o;
  o.device = c->device;
  o.input_dtype = c->input_dtype;
  o.normalize = c->normalize;
  o.stream = c->stream;
  ic_cache* child = ic_cache_create_ex(c->dim, K, &o);
  if (!child) return IC_ERR_NOMEM;   // message already set
  cudaError_t e = cudaMemcpyAsync(c->idx_init.p, init.data(), (size_t)K * 8, cudaMemcpyHostToDevice, c->stream);
  if (e == cudaSuccess)
    e = icc::launch_gather_rows(c->slab, static_cast<const int64_t*>(c->idx_init.p), (int)K, c->dim, child->slab,
                                child->ids, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // `init` is a host vector about to go away
  if (e != cudaSuccess) {
    ic_cache_destroy(child);
    return fail(IC_ERR_CUDA, "centroid seeding failed: %s", cudaGetErrorString(e));
  }
  child->size = K;
  child->launches += 1;
  // one status word for parent and child: a bounded wait that expires in a kernel launched through
  // the child (assignment passes, a query's centroid step) is reported by the parent's calls
  if (child->h_status) cudaFreeHost(child->h_status);
  child->h_status = nullptr;
  child->d_status = c->d_status;
  int64_t* assign = static_cast<int64_t*>(c->idx_assign.p);
  for (int it = 0; it <= n_iters && rc == IC_OK; ++it) {
    // assignment: every cached row is a query against the centroids, best centroid per row
    rc = query_bf16_rows(child, static_cast<const char*>(c->slab), n, c->capacity, 1, assign,
                         static_cast<float*>(c->idx_best.p), -1);
    if (rc != IC_OK) break;
    e = icc::launch_sort_by_cluster(assign, n, (int)K, static_cast<int*>(c->idx_sort.p),
                                    static_cast<int*>(c->idx_offsets.p), static_cast<int*>(c->idx_order.p), c->stream);
    if (e == cudaSuccess && it < n_iters)
      e = icc::launch_centroid_update(c->slab, c->dim, static_cast<const int*>(c->idx_offsets.p),
                                      static_cast<const int*>(c->idx_order.p), (int)K, child->slab, c->stream);
    if (e != cudaSuccess) rc = fail(IC_ERR_CUDA, "clustering launch failed: %s", cudaGetErrorString(e));
    child->launches += it < n_iters ? 5 : 4;
  }
  // Cluster-contiguous copy of the rows, so that a probed cluster is one contiguous run to stream.
  // It costs as much memory again as the indexed rows; when that is not to be had the search
  // fetches rows through the member lists instead (slower, same results).
  c->have_idx_rows = false;
  if (rc == IC_OK) {
    if (ensure(c, c->idx_rows, (size_t)n * c->dim * 2, "cluster-contiguous rows") == IC_OK) {
      e = icc::launch_gather_by_order(c->slab, static_cast<const int*>(c->idx_order.p), n, c->dim, c->idx_rows.p, c->stream);
      if (e != cudaSuccess) rc = fail(IC_ERR_CUDA, "row gather launch failed: %s", cudaGetErrorString(e));
      else c->have_idx_rows = true;
      child->launches += 1;
    } else {
      g_err[0] = 0;
    }
  }
  if (rc == IC_OK && cudaStreamSynchronize(c->stream) != cudaSuccess) rc = fail(IC_ERR_CUDA, "clustering failed on the device");
  if (rc == IC_OK) rc = check_timeout(c);
  if (rc != IC_OK) {
    char keep[sizeof g_err];
    memcpy(keep, g_err, sizeof keep);
    ic_cache_destroy(child);
    memcpy(g_err, keep, sizeof keep);
    return rc;
  }
  c->centroids = child;
  c->n_clusters = (int32_t)K;
  c->n_indexed = n;
  return IC_OK;
}

int ic_cache_index_info(const ic_cache_t* c, int32_t* n_clusters, int64_t* n_indexed) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (n_clusters) *n_clusters = c->n_clusters;
  if (n_indexed) *n_indexed = c->n_indexed;
  return IC_OK;
}

int ic_cache_read_index(ic_cache_t* c, void* centroids_host, int64_t* assign_host) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (!c->centroids) return fail(IC_ERR_INVALID, "no index: call ic_cache_build_index first");
  DeviceGuard guard(c->device);
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e == cudaSuccess && centroids_host)
    e = cudaMemcpy(centroids_host, c->centroids->slab, (size_t)c->n_clusters * c->dim * 2, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess && assign_host)
    e = cudaMemcpy(assign_host, c->idx_assign.p, (size_t)c->n_indexed * 8, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "index copy failed: %s", cudaGetErrorString(e));
  return IC_OK;
}

int ic_cache_query_clustered(ic_cache_t* c, const void* q, int32_t nq, int32_t k, int32_t nprobe, int64_t* out_ids,
                             float* out_scores, int64_t* out_probes) {
  int rc = check_query_args(c, q, nq, k, out_ids, out_scores);
  if (rc != IC_OK || nq == 0) return rc;
  if (!c->centroids) return fail(IC_ERR_INVALID, "no index: call ic_cache_build_index first");
  if (nprobe < 1 || nprobe > IC_MAX_PROBES) return fail(IC_ERR_INVALID, "nprobe %d outside [1, %d]", nprobe, IC_MAX_PROBES);
  DeviceGuard guard(c->device);
  if (!is_device_ptr(q, c->device) || !is_device_ptr(out_ids, c->device) || !is_device_ptr(out_scores, c->device) ||
      (out_probes && !is_device_ptr(out_probes, c->device)))
    return fail(IC_ERR_INVALID, "q, out_ids, out_scores and out_probes must be device pointers on device %d", c->device);
  if ((rc = check_timeout(c)) != IC_OK) return rc;
  const int np = nprobe;   // probes past the number of clusters come back as -1 and give empty lists
  const size_t q_row = (size_t)c->dim * in_elem_bytes(c);
  const int merge_lists_max = (c->smem_optin - 4096) / (k * 8 + 4);
  for (int q0 = 0; q0 < nq; q0 += WINDOW_MAX_NQ) {
    const int w = std::min(WINDOW_MAX_NQ, nq - q0);
    const char* qw = static_cast<const char*>(q) + (size_t)q0 * q_row;
    // pieces per probed cluster: about six CTAs per SM (the scan is latency-bound per CTA), pieces
    // of at least ~64 rows; the rows inserted since the build are cut into pieces of ~2048
    const int64_t avg_cluster = std::max<int64_t>(1, c->n_indexed / c->n_clusters);
    int n_split = (int)std::max<int64_t>(1, std::min<int64_t>({16, (6 * c->sm_count + (int64_t)w * np - 1) / ((int64_t)w * np),
                                                                avg_cluster / 64}));
    // Streaming the probed clusters from the cluster-contiguous copy pays from a few dozen (query,
    // probe) pairs on: pieces of at least ~256 rows, two CTAs per SM.
    int stream_split = 0, stream_stages = 0;
    if (c->have_idx_rows && c->dim <= 1024 && (int64_t)w * np >= 32) {
      // about four waves of CTAs (two per SM), so that the last wave's idle SMs cost little
      stream_split = (int)std::max<int64_t>(1, std::min<int64_t>({16, (8 * c->sm_count + (int64_t)w * np - 1) / ((int64_t)w * np),
                                                                   avg_cluster / 256}));
      const int half = c->smem_optin / 2 - 2048;
      stream_stages = 2;
      while (stream_stages < 4 && icc::cluster_stream_smem_bytes(c->dim, k, stream_stages + 1) <= half) ++stream_stages;
      if (icc::cluster_stream_smem_bytes(c->dim, k, stream_stages) > c->smem_optin) stream_split = 0;
      else n_split = stream_split;
    }
    // Rows inserted since the build are one contiguous range that every query scans: from a
    // thousand rows on, the tiles that lie wholly past the index go to the tensor-core kernel (one
    // launch over that tile range, its per-CTA lists joining the final merge; measured with
    // 200,000 such rows: 843 -> about 60 us for one query) and only the ragged head of the range
    // (fewer than 256 rows) stays with the cluster scan.
    const int64_t tile_lo = (c->n_indexed + ROW_TILE - 1) / ROW_TILE;
    const int64_t dense_rows = c->size - tile_lo * ROW_TILE;
    ic_cache_plan_t tpl;
    bool dense_tail = c->have_tmap_slab && dense_rows >= DENSE_TAIL_MIN_ROWS &&
                      plan_impl(c->dim, c->size, w, k, IC_PATH_UMMA, c->sm_count, c->smem_optin, &tpl) == IC_OK &&
                      np + 1 + tpl.n_partitions <= merge_lists_max;
    const int64_t scan_end = dense_tail ? std::min<int64_t>(c->size, tile_lo * ROW_TILE) : c->size;   // cluster scan covers [n_indexed, scan_end)
    const int64_t scan_tail = scan_end - c->n_indexed;
    const int dense_lists = dense_tail ? tpl.n_partitions : 0;
    int n_tail = scan_tail > 0 ? (int)std::max<int64_t>(1, std::min<int64_t>(32, (scan_tail + 2047) / 2048)) : 0;
    const int merge_lists_max_scan = merge_lists_max - dense_lists;
    while (np * n_split + n_tail > merge_lists_max_scan && n_split > 1) --n_split;
    if (np * n_split + n_tail > merge_lists_max_scan)
      n_tail = std::min(n_tail, std::max(scan_tail > 0 ? 1 : 0, merge_lists_max_scan - np * n_split));
    if (np * n_split + n_tail > merge_lists_max_scan)
      return fail(IC_ERR_UNSUPPORTED, "nprobe %d with k %d needs more partial lists than the merge kernel holds", nprobe, k);
    const int n_lists = np * n_split + n_tail;
    if ((rc = ensure(c, c->idx_probes, (size_t)w * nprobe * 8, "probed clusters")) != IC_OK) return rc;
    if ((rc = ensure(c, c->idx_probe_scores, (size_t)w * nprobe * 4, "centroid scores")) != IC_OK) return rc;
    const int nq_pad = (w + QUERY_TILE - 1) / QUERY_TILE * QUERY_TILE;
    if ((rc = ensure(c, c->q_bf16, (size_t)nq_pad * c->dim * 2, "query staging (bf16)")) != IC_OK) return rc;
    if ((rc = ensure(c, c->q_f32, (size_t)w * c->dim * 4, "query staging (fp32)")) != IC_OK) return rc;
    if ((rc = ensure(c, c->partials, (size_t)(n_lists + dense_lists) * w * k * 8, "partial top-k lists")) != IC_OK) return rc;
    // centroid step: the nprobe best centroids of every query (labels = cluster numbers); past
    // the number of clusters the rows are padded with -1
    int64_t* probes = out_probes ? out_probes + (size_t)q0 * nprobe : static_cast<int64_t*>(c->idx_probes.p);
    rc = do_query_window(c->centroids, qw, w, nprobe, probes, static_cast<float*>(c->idx_probe_scores.p), -INFINITY, nullptr);
    if (rc != IC_OK) return rc;
    // the same bf16-rounded queries, widened to fp32, for the scan of the clusters
    cudaError_t e = icc::launch_convert_rows(qw, c->input_dtype == IC_F32, w, c->dim, c->normalize, c->q_bf16.p,
                                             static_cast<float*>(c->q_f32.p), nq_pad, nullptr, nullptr, c->stream);
    // The probed clusters: with the cluster-contiguous copy and enough (query, probe) pairs to fill
    // the GPU, one bulk-copy pipeline per piece (two CTAs per SM); otherwise the register-load kernel,
    // which also takes the ragged rows past the index.
    const bool stream = c->have_idx_rows && c->dim <= 1024 && stream_split > 0;
    if (e == cudaSuccess && stream) {
      icc::ClusterStreamParams cp;
      cp.sorted_rows = c->idx_rows.p;
      cp.dim = c->dim;
      cp.q_f32 = static_cast<const float*>(c->q_f32.p);
      cp.nq = w;
      cp.k = k;
      cp.probes = probes;
      cp.n_probe = nprobe;
      cp.n_split = n_split;
      cp.offsets = static_cast<const int*>(c->idx_offsets.p);
      cp.order = static_cast<const int*>(c->idx_order.p);
      cp.partials = static_cast<uint64_t*>(c->partials.p);
      cp.n_stages = stream_stages;
      cp.smem_bytes = icc::cluster_stream_smem_bytes(c->dim, k, stream_stages);
      cp.dev_status = c->d_status;
      e = icc::launch_cluster_stream(cp, c->stream);
      c->launches += 1;
    }
    if (e == cudaSuccess)
      e = icc::launch_cluster_scan(c->slab, c->have_idx_rows ? c->idx_rows.p : nullptr, scan_end, c->dim,
                                   static_cast<const float*>(c->q_f32.p), w, k, probes, nprobe, n_split, n_tail,
                                   static_cast<const int*>(c->idx_offsets.p), static_cast<const int*>(c->idx_order.p),
                                   c->n_indexed, static_cast<uint64_t*>(c->partials.p), stream ? np * n_split : 0, c->stream);
    if (e != cudaSuccess) return fail(IC_ERR_CUDA, "two-level search launch failed: %s", cudaGetErrorString(e));
    if (dense_tail) {
      int unused = 0;
      rc = run_umma_passes(c, tpl, c->q_bf16.p, w, nq_pad, k, static_cast<uint64_t*>(c->partials.p) + (size_t)n_lists * w * k,
                           nullptr, nullptr, static_cast<unsigned long long*>(c->pace.p), &unused, false, tile_lo);
      if (rc != IC_OK) return rc;
    }
    e = icc::launch_merge(static_cast<const uint64_t*>(c->partials.p), n_lists + dense_lists, w, k, c->ids,
                          out_ids + (size_t)q0 * k, out_scores + (size_t)q0 * k, -INFINITY, nullptr, c->stream);
    if (e != cudaSuccess) return fail(IC_ERR_CUDA, "two-level search launch failed: %s", cudaGetErrorString(e));
    c->launches += 3;
  }
  return IC_OK;
}

int ic_cache_probe_wait_limit(ic_cache_t* c) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  DeviceGuard guard(c->device);
  cudaError_t e = icc::launch_wait_limit_probe(2000000ll /* about a millisecond */, c->d_status, c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "probe launch failed: %s", cudaGetErrorString(e));
  c->launches += 1;
  return IC_OK;
}

int ic_cache_set_stream(ic_cache_t* c, void* cuda_stream) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  if (c->centroids) c->centroids->stream = c->stream;
  return IC_OK;
}

int ic_cache_set_path(ic_cache_t* c, int32_t path) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  if (path < IC_PATH_AUTO || path > IC_PATH_UMMA) return fail(IC_ERR_INVALID, "unknown path %d", path);
  c->forced_path = path;
  return IC_OK;
}

int64_t ic_cache_size(const ic_cache_t* c) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  return c->size;
}

int ic_cache_clear(ic_cache_t* c) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  c->size = 0;
  if (c->centroids) {
    DeviceGuard guard(c->device);
    drop_index(c);   // (synchronises the stream)
  }
  return IC_OK;
}

int ic_cache_sync(ic_cache_t* c) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  DeviceGuard guard(c->device);
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "stream sync failed: %s", cudaGetErrorString(e));
  if (c->h_status && *reinterpret_cast<volatile int*>(c->h_status) != 0) {
    const int code = *c->h_status;
    *c->h_status = 0;
    return fail(IC_ERR_TIMEOUT, code == 3 ? "a kernel failed a debug-build index check (code %d); its results are suspect"
                                          : "a kernel gave up on a bounded wait (code %d); its results are incomplete", code);
  }
  return IC_OK;
}

int ic_cache_set_profiling(ic_cache_t* c, int32_t enable) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  c->profiling = enable != 0;
  return IC_OK;
}

int ic_cache_read_profile(ic_cache_t* c, double* scoring_ms, int64_t* scoring_launches, double* merge_ms,
                          int64_t* merge_launches, double* seed_ms, int64_t* seed_passes) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  DeviceGuard guard(c->device);
  cudaError_t e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) return fail(IC_ERR_CUDA, "stream sync failed: %s", cudaGetErrorString(e));
  double sums[3] = {0.0, 0.0, 0.0};
  int64_t counts[3] = {0, 0, 0};
  std::vector<cudaEvent_t>* pools[3] = {&c->ev_score, &c->ev_merge, &c->ev_seed};
  size_t* used[3] = {&c->n_ev_score, &c->n_ev_merge, &c->n_ev_seed};
  for (int w = 0; w < 3; ++w) {
    for (size_t i = 0; i + 1 < *used[w]; i += 2) {
      float ms = 0.0f;
      if (cudaEventElapsedTime(&ms, (*pools[w])[i], (*pools[w])[i + 1]) == cudaSuccess) {
        sums[w] += ms;
        counts[w] += 1;
      } else {
        cudaGetLastError();
      }
    }
    *used[w] = 0;
  }
  if (scoring_ms) *scoring_ms = sums[0];
  if (scoring_launches) *scoring_launches = counts[0];
  if (merge_ms) *merge_ms = sums[1];
  if (merge_launches) *merge_launches = counts[1];
  if (seed_ms) *seed_ms = sums[2];
  if (seed_passes) *seed_passes = counts[2];
  return IC_OK;
}

int64_t ic_cache_launch_count(const ic_cache_t* c) {
  if (!c) return fail(IC_ERR_INVALID, "NULL handle");
  return c->launches + (c->centroids ? c->centroids->launches : 0);
}

}  // extern "C"
