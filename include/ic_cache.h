/*
 * ic_cache.h - C ABI of the B200 example-retrieval library.
 *
 * The library implements stage 1 of IC-Cache's example selection: keep one dense embedding
 * per cached request and, for each batch of incoming request embeddings, return the k cached
 * examples with the highest cosine similarity, with their ids and scores (paper Sec. 4.1,
 * "Two-Stage Scalable Example Selection"; Algorithm 1, RetrieveExamples stage 1,
 * GetSimilarExamples(request_emb, examples)).  Registration of a served request
 * (client.update_cache in the client listing of Sec. 3; step 4 of the overview figure) is
 * ic_cache_insert.
 *
 * Storage: a row-major bf16 slab [capacity, dim] in device memory plus an int64 id per row.
 * Scores are inner products of the stored bf16 rows with the bf16-rounded query, accumulated
 * in fp32; they equal cosine similarity when inputs are unit vectors or `normalize` is set.
 *
 * Conventions common to all calls
 *   - Unless a call says "host", every data pointer is a DEVICE pointer on the handle's
 *     device, dense and row-major.  The caller owns those buffers; the library never frees
 *     or retains them past the work it enqueues.
 *   - insert/query validate on the host, enqueue kernels on the handle's stream and return
 *     without synchronising.  Outputs are valid once that stream has reached the call.  A
 *     query enqueued after an insert on the same stream sees the inserted rows.
 *   - One handle is bound to one stream and is not thread-safe; handles are independent.
 *   - Every call returns IC_OK or a negative ic_status.  On a non-OK return nothing was
 *     enqueued and the cache is unchanged (an insert is all-or-nothing).  The paper's
 *     fault-tolerance rule (Sec. 5, "Fault Tolerance": bypass the retriever when it fails)
 *     maps to: treat any non-OK status as "serve without examples".
 *   - There is no CPU fallback: without a CUDA device ic_cache_create fails.
 */
#ifndef IC_CACHE_H_
#define IC_CACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ic_cache ic_cache_t; /* opaque, owned by the library */

enum ic_status {
  IC_OK = 0,
  IC_ERR_INVALID = -1,     /* bad argument (NULL pointer, bad dim/k/count, host pointer) */
  IC_ERR_NOMEM = -2,       /* device allocation failed or caller workspace too small     */
  IC_ERR_FULL = -3,        /* insert would exceed capacity                                */
  IC_ERR_CUDA = -4,        /* CUDA runtime/driver error, or no usable device              */
  IC_ERR_UNSUPPORTED = -5, /* shape outside what the forced kernel path supports          */
  IC_ERR_TIMEOUT = -6      /* a bounded device-side wait expired in an earlier launch     */
};

enum ic_dtype { IC_BF16 = 0, IC_F32 = 1 };

/* Kernel path used for scoring (see ic_cache_plan). */
enum ic_path {
  IC_PATH_AUTO = 0,    /* scan for one or two queries (512 <= dim <= 1024), tensor cores otherwise */
  IC_PATH_GENERIC = 1, /* plain CUDA-core kernel, any shape; slow, kept as a cross-check  */
  IC_PATH_SCAN = 2,    /* bulk-copy staged CUDA-core scan, nq <= 4 per pass, dim <= 1024  */
  IC_PATH_UMMA = 3     /* tcgen05 tensor-core tiles with the top-k fused in the epilogue  */
};

#define IC_MAX_K 128        /* largest k accepted by ic_cache_query                         */
#define IC_MAX_DIM 4096     /* largest embedding dimension; dim must be a multiple of 8     */

/* Options for ic_cache_create_ex.  Zero-initialise, set struct_size = sizeof, then fill. */
typedef struct ic_cache_opts {
  uint32_t struct_size; /* sizeof(ic_cache_opts_t) of the caller's build                   */
  int32_t device;       /* CUDA device ordinal; -1 = the current device                    */
  int32_t input_dtype;  /* ic_dtype of the emb and q pointers (default IC_BF16)            */
  int32_t normalize;    /* 1: L2-normalise rows on insert and queries on query (fp32)      */
  void* slab;           /* optional caller-owned device buffer, capacity*dim*2 bytes,
                           256-byte aligned; NULL = the library allocates                  */
  void* ids;            /* optional caller-owned device buffer, capacity*8 bytes           */
  void* stream;         /* cudaStream_t; NULL = the legacy default stream                  */
  void* workspace;      /* optional caller-owned device buffer (256-byte aligned) that serves
                           as the scratch of ic_cache_query / ic_cache_query_min_score, which
                           then allocate nothing; NULL = the library grows its own buffers   */
  size_t workspace_bytes; /* its size; see ic_cache_workspace_bytes                          */
} ic_cache_opts_t;

/* Host-side launch plan for one query call; pure function of its arguments. */
typedef struct ic_cache_plan {
  int32_t path;          /* ic_path actually used                                          */
  int32_t query_tile;    /* queries handled together by one CTA (tensor cores: 128, or 64
                            with a resident query tile)                                    */
  int32_t n_query_tiles; /* per launch                                                     */
  int32_t n_partitions;  /* row partitions = partial top-k lists per query                 */
  int32_t n_ctas;        /* CTAs of the scoring kernel                                     */
  int32_t n_stages;      /* shared-memory ring stages (0 for the generic path)             */
  int32_t smem_bytes;    /* dynamic shared memory of the scoring kernel                    */
  int32_t n_launches;    /* scoring launches needed for the whole batch                    */
  int32_t queue_cap;     /* tensor-core path: candidate queue entries per query (else 0)   */
  int32_t seed_tiles;    /* tensor-core path: 256-row tiles scored into lists ahead of the
                            main pass, whose merged k-th key is the main pass's floor; the
                            main pass skips them (0 = none)                                */
  int32_t seed0_tiles;   /* tensor-core path: tiles (the first few of every partition, about
                            one per SM in all, more in a long sampling launch) whose group
                            maxima the CTAs of a launch exchange to agree on a first floor
                            per query (0 = no seeding inside the launch)                   */
  int32_t cta_group;     /* tensor-core path: 2 = CTA pairs issue one 256-query MMA and
                            split each row tile between them, 1 = single CTAs (else 0)     */
  int32_t query_resident;/* tensor-core path: 1 = at most 64 queries, M = 64, the whole query
                            tile stays in shared memory and ring stages hold cache rows only */
} ic_cache_plan_t;

/*
 * Create an empty cache for embeddings of `dim` components with room for `capacity` entries
 * on the current device, input dtype bf16, no normalisation, legacy default stream.  (Paper:
 * the example cache that IC-Cache's Example Manager owns, Sec. 3 overview and Sec. 4.3; the pool
 * `examples` that Algorithm 1's GetSimilarExamples searches.  The paper bounds the cache by a
 * capacity and evicts when it is full; here the capacity is fixed at creation.)
 * dim: multiple of 8, 8 <= dim <= IC_MAX_DIM.  capacity: 1 .. 2^31 - 512.
 * Returns NULL on failure; ic_cache_last_error() then describes why.
 */
ic_cache_t* ic_cache_create(int32_t dim, int64_t capacity);

/* As ic_cache_create, with options (NULL opts = defaults).  Buffers passed in opts are
 * borrowed and must outlive the handle. */
ic_cache_t* ic_cache_create_ex(int32_t dim, int64_t capacity, const ic_cache_opts_t* opts);

/*
 * Append n embeddings and their ids at slots [size, size+n) (paper: update_cache after the
 * response is served).  emb: [n, dim] in the handle's input dtype; fp32 is rounded to bf16,
 * round-to-nearest-even, after the optional fp32 L2 normalisation (a zero row stays zero).
 * ids: [n] int64, opaque to the library, not checked for uniqueness.
 * n == 0 is a no-op.  IC_ERR_FULL if size + n > capacity, IC_ERR_INVALID for n < 0 or a NULL
 * or host pointer with n > 0.
 */
int ic_cache_insert(ic_cache_t* c, const void* emb, const int64_t* ids, int64_t n);

/*
 * For each of nq query embeddings return the k entries with the largest score.  (Paper:
 * Algorithm 1, RetrieveExamples stage 1, GetSimilarExamples(request_emb, examples): the
 * relevance stage of Sec. 4.1, which ranks cached examples by the cosine similarity of dense
 * request embeddings, best first; the result is the candidate set handed to the stage-2 proxy.)
 * q: [nq, dim] in the handle's input dtype (rounded to bf16 like inserted rows).
 * out_ids [nq, k] int64, out_scores [nq, k] fp32: each row sorted by score descending, equal
 * scores ordered by earlier insertion; when k exceeds the number of entries the tail is
 * id -1, score -infinity.  1 <= k <= IC_MAX_K; nq == 0 is a no-op.
 * Every score comes from an exhaustive pass over all entries: the result is the exact top-k
 * of the fp32-accumulated scores (no clustering or other approximation).
 * May grow the library's scratch buffers on the first call with a larger nq or k (this
 * synchronises the stream); later calls of the same or smaller shape allocate nothing.
 */
int ic_cache_query(ic_cache_t* c, const void* q, int32_t nq, int32_t k, int64_t* out_ids,
                   float* out_scores);

/*
 * Bytes of workspace (ic_cache_opts_t.workspace) that ic_cache_query needs at most for batches
 * of up to max_nq queries and k up to max_k against up to `capacity` entries of dimension dim,
 * on the current CUDA device (the launch plan depends on its SM count; without a device the
 * figures of a B200 are used).  0 for invalid arguments.  With a workspace the handle's
 * queries take all scratch (query staging, partial lists, floors, group maxima) from it and
 * return IC_ERR_NOMEM, enqueuing nothing, when a call needs more than it holds; the other
 * calls (host variants, self-similarity, index, removal) still use library-owned buffers.  Like
 * the static scratch, a workspace must not be shared by calls that overlap on the GPU.
 */
size_t ic_cache_workspace_bytes(int32_t dim, int64_t capacity, int32_t max_nq, int32_t max_k);

/*
 * ic_cache_query that reports only entries whose score reaches min_score: the hit test of
 * semantic caching (paper Sec. 2.2: reuse a cached response when the most similar request is
 * similar enough; its evaluation's similarity-threshold baselines) and a similarity pre-filter
 * in front of the utility threshold of Sec. 4.1.  Same arguments, order and padding as
 * ic_cache_query; entries of the top-k scoring below min_score are returned as id -1, score
 * -infinity.  out_counts: optional device array [nq] of int32 receiving how many entries
 * each query kept (0 .. min(k, size)); NULL to skip.  min_score = -infinity keeps everything;
 * NaN is IC_ERR_INVALID.
 */
int ic_cache_query_min_score(ic_cache_t* c, const void* q, int32_t nq, int32_t k, float min_score,
                             int64_t* out_ids, float* out_scores, int32_t* out_counts);

/*
 * ic_cache_query for callers whose buffers live in HOST memory (pinned memory makes the
 * copies asynchronous): copies q to the device, runs the query, copies both results back
 * and synchronises the stream before returning.
 */
int ic_cache_query_host(ic_cache_t* c, const void* q_host, int32_t nq, int32_t k,
                        int64_t* out_ids_host, float* out_scores_host);

/*
 * ic_cache_query without any allocation (the paper has no counterpart; this exists for
 * deployment).  Some callers must not allocate device memory at query time: a serving
 * process whose framework has already reserved the whole GPU for its own memory pool (so a
 * late cudaMalloc fails), or a latency-critical loop whose rules forbid calls that may
 * synchronise the device, which cudaMalloc and cudaFree do.  ic_cache_query grows the
 * library's scratch buffers on the first call of a larger shape; this variant never does.
 * Its scratch (query staging, partial top-k lists, seed thresholds, group maxima, progress words) is carved out of one
 * fixed array of IC_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that
 * loads the library holds that much memory until the process exits, whether or not this
 * call is ever used.
 *
 * Arguments, results and ordering are exactly those of ic_cache_query (device pointers).
 * Differences:
 *   - a query whose scratch need exceeds IC_STATIC_SCRATCH_BYTES returns IC_ERR_NOMEM and
 *     enqueues nothing; nq above 1024 returns IC_ERR_INVALID.  The need is about
 *     6*dim*nq bytes of query staging plus 8*k*nq bytes per partial list, with up to
 *     2*(SM count / ceil(nq/128)) + 1 lists; 64 queries, k = 10, dim = 768 need about 2 MB.
 *   - the first call on a device looks up the array's device address (once per device, with
 *     that device current); make that first call outside any stream capture.
 *   - every handle, stream and thread of the process shares the one array per GPU, and it
 *     keeps the previous call's contents.  A call writes every data word (staged queries, lists,
 *     floors, maxima) before it reads it, and the few progress and completion words that CTAs
 *     of one launch exchange carry a launch number drawn from one counter for the whole
 *     process, so a word left by an earlier call, of this or any other handle, is never taken
 *     for a current one: nothing needs clearing.  But two calls whose kernels overlap on the GPU
 *     (different streams or handles) race on the scratch and return garbage: keep them ordered.
 *   - it calls no cudaMalloc, cudaFree, event creation or other allocating routine, and
 *     ignores ic_cache_set_profiling.
 */
#define IC_STATIC_SCRATCH_BYTES (8u << 20)
int ic_cache_query_static(ic_cache_t* c, const void* q, int32_t nq, int32_t k, int64_t* out_ids,
                          float* out_scores);

/*
 * ic_cache_insert for HOST buffers: copies rows and ids to the device (in slices of at most
 * 64 MiB) and enqueues the insert.  Returns once everything is enqueued; pageable buffers may be
 * reused at once, PINNED buffers must stay unchanged until a synchronising call
 * (ic_cache_query_host, ic_cache_sync) has returned.
 */
int ic_cache_insert_host(ic_cache_t* c, const void* emb_host, const int64_t* ids_host, int64_t n);

/*
 * Similarity of cached entries to the OTHER cached entries (the request-similarity study of
 * paper Sec. 2.2: each request's best match among the other requests).  For each of the `count`
 * entries in slots [first, first+count): the id and score of the best-scoring entry other than
 * itself (an exact copy of it counts as another entry; ties go to the lower slot).
 * out_ids [count] int64, out_scores [count] fp32, device pointers; (-1, -infinity) when the
 * cache holds a single entry.  The stored bf16 rows serve as the queries; work is
 * count * size * dim multiply-adds on the tensor-core path, in passes of 1024 entries.
 * Stream-ordered like ic_cache_query; may grow scratch on first use.
 */
int ic_cache_self_similarity(ic_cache_t* c, int64_t first, int64_t count, int64_t* out_ids,
                             float* out_scores);

/*
 * Eviction mechanics (paper Sec. 4.3, "Example Manager": a background solver picks the
 * examples to drop when the cache is full; which ones is the caller's policy).  Removes every
 * entry whose id equals one of ids_host[0..n) (HOST array; ids that match nothing are
 * ignored) and closes the gaps: surviving entries from the end of the slab move, in order,
 * into the vacated slots, so size shrinks by the number removed and capacity is free again
 * for ic_cache_insert.  After a removal "equal scores are ordered by earlier insertion"
 * reads "by lower slot": a moved entry ranks among equal scores by its new position.
 * *n_removed (optional) receives the number of entries removed.  Synchronises the stream.
 * Not part of the per-request path: one pass over the id array (8 bytes per entry) plus the
 * moved rows.  IC_ERR_UNSUPPORTED if more than 4n + 1024 entries carry the given ids.
 */
int ic_cache_remove(ic_cache_t* c, const int64_t* ids_host, int64_t n, int64_t* n_removed);

/*
 * Checkpoint and restore (paper Sec. 5, "Fault Tolerance": every component periodically
 * checkpoints its state).  ic_cache_save writes the entries (stored bf16 rows, ids, utilities if
 * any) to a file on the HOST file system; ic_cache_load replaces the handle's contents with a
 * file written by ic_cache_save for the same dimension (size at most this handle's capacity),
 * keeping slots, ids and utilities, so queries return exactly what they returned before.  Both
 * synchronise the stream and copy through host memory; neither is part of the per-request path.
 * The two-level index is not stored: rebuild it after loading.  On a failed load the handle is
 * left empty.  IC_ERR_INVALID for an unreadable, foreign or mismatching file.
 */
int ic_cache_save(ic_cache_t* c, const char* path);
int ic_cache_load(ic_cache_t* c, const char* path);

/*
 * Per-entry utility for the cache-management policy (paper Sec. 4.3, "Example Manager": each
 * example's value is the efficiency gain it enabled, i.e. the number of successful offloadings,
 * kept as a moving average that is multiplied by 0.9 every hour; a knapsack solver run by the
 * caller decides what to evict).  The library keeps one fp32 utility per entry, 0 for a new entry;
 * it moves with the entry when ic_cache_remove closes gaps.  The array (4 bytes per slot of
 * capacity) is allocated by the first ic_cache_utility_add.
 *
 * ic_cache_utility_add: for i in 0..n-1, in order, add gains_host[i] (finite) to the utility of
 * every entry whose id is ids_host[i] (HOST arrays; ids that match nothing are ignored; one fp32
 * addition per match).  One pass over the id array; synchronises the stream.
 * ic_cache_utility_decay: multiply every entry's utility by factor (finite, >= 0; 0.9 per hour in
 * the paper; the caller owns the clock).  Stream-ordered.
 * ic_cache_utility_read: copy ids and utilities of slots 0 .. size-1 to HOST arrays (either may
 * be NULL) for the caller's solver, which then calls ic_cache_remove.  Synchronises the stream.
 */
int ic_cache_utility_add(ic_cache_t* c, const int64_t* ids_host, const float* gains_host, int64_t n);
int ic_cache_utility_decay(ic_cache_t* c, float factor);
int ic_cache_utility_read(ic_cache_t* c, int64_t* ids_host, float* utility_host);

/*
 * Two-level search (paper Sec. 4.1, "Two-Stage Scalable Example Selection": cached examples
 * are clustered offline into K groups with K-Means, K = sqrt(N) balancing the K centroid
 * comparisons against the N/K comparisons inside a cluster; a request is matched to centroids
 * first and searched inside the closest clusters).
 *
 * ic_cache_build_index clusters the entries present at the time of the call.  The paper only
 * names K-Means; here it is Lloyd iteration under the retrieval metric: an entry belongs to
 * the centroid with the largest score (ties: lower centroid number), a centroid is the mean of
 * its entries scaled to unit length and stored as bf16.  n_clusters: 0 = round(sqrt(size)),
 * else 1 .. min(size, IC_MAX_CLUSTERS).  n_iters >= 0 update steps (0 keeps the initial
 * centroids).  init_slots_host: HOST array of n_clusters distinct slots whose rows are the
 * initial centroids, or NULL for slots floor(c * size / n_clusters).  Entries are not moved:
 * slots, ids and the results of ic_cache_query are unaffected.  The index keeps its own copy of the
 * indexed rows in cluster order (size * dim * 2 bytes more device memory) so that a probed cluster
 * is one contiguous run to read; if that allocation fails the search reads rows through the member
 * lists instead (slower, same results).  Not part of the per-request
 * path (each iteration scores every entry against every centroid and reads the slab once
 * more); synchronises the stream.  Replaces any earlier index.  ic_cache_remove and
 * ic_cache_clear drop the index; entries inserted later stay outside it and are searched
 * exhaustively by every ic_cache_query_clustered until the index is rebuilt.
 */
#define IC_MAX_CLUSTERS 16384
#define IC_MAX_PROBES 64
int ic_cache_build_index(ic_cache_t* c, int32_t n_clusters, int32_t n_iters, const int64_t* init_slots_host);

/* Number of clusters of the current index (0 = none) and number of entries it covers.  Either
 * output may be NULL. */
int ic_cache_index_info(const ic_cache_t* c, int32_t* n_clusters, int64_t* n_indexed);

/* Copy the index to HOST buffers (inspection and tests): centroids_host [n_clusters, dim] bf16
 * bit patterns, assign_host [n_indexed] int64 cluster of each indexed slot.  Either may be NULL.
 * Synchronises the stream.  IC_ERR_INVALID without an index. */
int ic_cache_read_index(ic_cache_t* c, void* centroids_host, int64_t* assign_host);

/*
 * ic_cache_query restricted to the entries of the nprobe clusters whose centroids score
 * highest for the query (ties: lower cluster number) plus every entry inserted after the index
 * was built.  An approximation of ic_cache_query by design: an entry of the true top-k that
 * sits in a cluster that is not probed is missed; with nprobe = n_clusters the results are
 * those of ic_cache_query.  Same argument conventions, ordering and padding as
 * ic_cache_query.  1 <= nprobe <= IC_MAX_PROBES (clamped to n_clusters); out_probes: optional
 * device array [nq, nprobe] int64 receiving the probed clusters, best first, -1 padded.
 * IC_ERR_INVALID without an index.  Work per query: n_clusters + the probed clusters' entries
 * (about nprobe * size / n_clusters) + the entries inserted since, instead of size.
 */
int ic_cache_query_clustered(ic_cache_t* c, const void* q, int32_t nq, int32_t k, int32_t nprobe,
                             int64_t* out_ids, float* out_scores, int64_t* out_probes);

/* Release the handle and everything the library allocated for it (synchronises the handle's
 * stream first; buffers lent through ic_cache_opts_t are left to the caller).  NULL is a no-op.
 * (Paper Sec. 5, "Fault Tolerance": the serving path keeps working without the retriever, so a
 * caller may destroy a handle that reported an error and serve without examples, or re-create
 * it and restore a checkpoint.) */
void ic_cache_destroy(ic_cache_t* c);

/* Bind the handle to another stream (a cudaStream_t; NULL = legacy default stream).  Work
 * already enqueued stays on the old stream; ordering between the two is the caller's. */
int ic_cache_set_stream(ic_cache_t* c, void* cuda_stream);

/* Force a kernel path for later queries (IC_PATH_AUTO restores the default choice).  A
 * query whose shape the forced path cannot serve returns IC_ERR_UNSUPPORTED. */
int ic_cache_set_path(ic_cache_t* c, int32_t path);

/* Number of entries inserted so far, or a negative ic_status for a NULL handle. */
int64_t ic_cache_size(const ic_cache_t* c);

/* Forget all entries (size becomes 0); the slab is not cleared.  Stream-ordered. */
int ic_cache_clear(ic_cache_t* c);

/* Synchronise the handle's stream and report IC_ERR_TIMEOUT if any kernel since the last
 * call of this function gave up on a bounded wait, IC_ERR_CUDA on a CUDA error, else IC_OK.
 * (The debug build of the library, libic_cache_debug.so, compiled with -DIC_CACHE_DEBUG_CHECKS,
 * additionally checks tile, list and slot indices on the device; a failed check is reported here
 * the same way, with a message that says so.  No build ever traps on the device.) */
int ic_cache_sync(ic_cache_t* c);

/*
 * Diagnostic for the failure path.  Every device-side wait in this library is bounded; this
 * call enqueues a one-thread kernel whose wait is made to run out after about a millisecond
 * (it waits for a barrier that nothing completes) and which then reports the expiry the way a
 * scoring kernel would.  Afterwards ic_cache_query / ic_cache_insert return IC_ERR_TIMEOUT
 * until ic_cache_sync has reported and cleared it; the cache contents are untouched and the
 * handle stays usable.  Lets a caller test its "serve without examples" bypass.
 */
int ic_cache_probe_wait_limit(ic_cache_t* c);

/* Kernels launched by this handle so far (insert, query preparation, scoring, merge). */
int64_t ic_cache_launch_count(const ic_cache_t* c);

/*
 * Measurement aid.  While enabled, the launches of this handle are bracketed by pairs of CUDA
 * events on the handle's stream, in three groups: "scoring" = the scan launch(es), or the main
 * pass of the tensor-core path (the launch that reads all rows outside the list-level sample);
 * "seed" = the launch that scores the list-level sample of a large cache together with the merge
 * that turns its lists into per-query floors; "merge" = the final merge.  At most 16384 brackets of each group between two reads; later ones go
 * unrecorded.  ic_cache_query_static records nothing.
 */
int ic_cache_set_profiling(ic_cache_t* c, int32_t enable);

/* Synchronise the stream and return the device time (ms) and number of brackets of each group
 * recorded since the previous read.  Any output pointer may be NULL. */
int ic_cache_read_profile(ic_cache_t* c, double* scoring_ms, int64_t* scoring_launches,
                          double* merge_ms, int64_t* merge_launches, double* seed_ms,
                          int64_t* seed_passes);

/*
 * The launch plan the library would use for a query of nq vectors, k results, over n entries
 * of dimension dim on a device with sm_count multiprocessors and smem_optin bytes of opt-in
 * shared memory per block.  path = IC_PATH_AUTO or a forced ic_path.  Touches no device.
 * Returns IC_OK, IC_ERR_INVALID or IC_ERR_UNSUPPORTED.
 */
int ic_cache_plan(int32_t dim, int64_t n, int32_t nq, int32_t k, int32_t path, int32_t sm_count,
                  int32_t smem_optin, ic_cache_plan_t* plan);

/* Message for the most recent failure on the calling thread ("" if none). */
const char* ic_cache_last_error(void);

/* Library version, major*10000 + minor*100 + patch. */
int32_t ic_cache_version(void);

#ifdef __cplusplus
}
#endif
#endif /* IC_CACHE_H_ */
