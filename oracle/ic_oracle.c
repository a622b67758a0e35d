/*
 * CPU oracle for IC-Cache stage-1 example retrieval.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product path links, imports or calls this file.  It shares no
 * code with the CUDA library.
 *
 * What it computes is the plain definition of the step, not an algorithm:
 *   - relevance of a cached example to a request = cosine similarity of their
 *     dense text embeddings (paper Sec. 4.1, "Example Selector", first paragraph;
 *     Sec. 2.2 similarity study: cosine, 1 = identical requests);
 *   - the relevance stage ranks cached examples by that similarity, best first
 *     (Sec. 4.1, two-stage selection paragraph) = return the k best-scoring
 *     cached examples;
 *   - Algorithm 1, RetrieveExamples stage 1: GetSimilarExamples(request_emb,
 *     examples).
 * Every score is a brute-force fp32 dot product with the terms added in index
 * order, and every query's ranking is a full sort of all n (score, slot) pairs
 * by score descending, then slot (insertion position) ascending.  No blocking,
 * no partial selection, no reordering.
 *
 * bf16 here is the published format: the upper 16 bits of an IEEE-754 binary32;
 * widening appends 16 zero bits, narrowing rounds to nearest, ties to even.
 *
 * Parity pins: tests/test_oracle_pins.py (hand-computed cases, invariants,
 * library cross-check, closed-form statistics); the K-Means and two-level search
 * functions at the end of this file are pinned in tests/test_oracle_clustered_pins.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_BF16 = 0, ORACLE_F32 = 1 };

float ic_oracle_bf16_to_f32(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

/* Round-to-nearest-even narrowing of binary32 to bf16.  NaN stays NaN (quiet). */
uint16_t ic_oracle_f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, sizeof u);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
  uint32_t kept_lsb = (u >> 16) & 1u;
  u += 0x7fffu + kept_lsb;
  return (uint16_t)(u >> 16);
}

/* Element j of a row stored as dtype, widened to fp32; optionally passed
 * through one bf16 rounding first (what a bf16 store keeps of an fp32 input). */
static float load_elem(const void* base, int dtype, int64_t idx, int round_bf16) {
  if (dtype == ORACLE_BF16) return ic_oracle_bf16_to_f32(((const uint16_t*)base)[idx]);
  float v = ((const float*)base)[idx];
  if (round_bf16) v = ic_oracle_bf16_to_f32(ic_oracle_f32_to_bf16(v));
  return v;
}

typedef struct {
  float score;
  int64_t slot;
} pair_t;

/* score descending, then slot ascending */
static int cmp_pair(const void* a, const void* b) {
  const pair_t* x = (const pair_t*)a;
  const pair_t* y = (const pair_t*)b;
  if (x->score > y->score) return -1;
  if (x->score < y->score) return 1;
  if (x->slot < y->slot) return -1;
  if (x->slot > y->slot) return 1;
  return 0;
}

/*
 * Scores of one query against all n rows: s[i] = sum_j q[j] * x[i][j], fp32,
 * j ascending.  With normalize != 0 the sum is divided by ||q|| * ||x_i||
 * (fp32 norms, same summation order); a zero norm gives score 0.
 * Rows are independent, so the outer loop may be split over `threads` host
 * threads; that changes no arithmetic.
 */
static void score_one_query(const void* X, int x_dtype, int64_t n, int32_t d, const float* q,
                            int normalize, int round_bf16, int threads, float* s) {
  float qn = 0.0f;
  if (normalize) {
    for (int32_t j = 0; j < d; ++j) qn += q[j] * q[j];
    qn = sqrtf(qn);
  }
  if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    float acc = 0.0f;
    float xn = 0.0f;
    for (int32_t j = 0; j < d; ++j) {
      float x = load_elem(X, x_dtype, i * (int64_t)d + j, round_bf16);
      acc += q[j] * x;
      if (normalize) xn += x * x;
    }
    if (normalize) {
      xn = sqrtf(xn);
      acc = (qn > 0.0f && xn > 0.0f) ? acc / (qn * xn) : 0.0f;
    }
    s[i] = acc;
  }
}

/*
 * Exhaustive top-k retrieval.
 *   X [n,d], Q [nq,d] row-major, dtype ORACLE_BF16 (uint16 bit patterns) or
 *   ORACLE_F32; ids [n] caller labels (NULL: id = slot).
 *   round_bf16: fp32 inputs are first rounded to bf16 (no effect on bf16 input).
 *   out_ids/out_scores/out_slots [nq,k] (out_slots may be NULL); rows past
 *   min(k,n) are padded with id -1, slot -1, score -inf.
 *   all_scores: NULL, or [nq,n] receiving every score (for acceptance checks).
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int ic_oracle_search(const void* X, int x_dtype, const int64_t* ids, int64_t n, int32_t d,
                     const void* Q, int q_dtype, int32_t nq, int32_t k, int normalize,
                     int round_bf16, int threads, int64_t* out_ids, float* out_scores,
                     int64_t* out_slots, float* all_scores) {
  if (n < 0 || d <= 0 || nq < 0 || k < 0) return -1;
  if ((n > 0 && !X) || (nq > 0 && !Q)) return -1;
  float* q = (float*)malloc(sizeof(float) * (size_t)d);
  float* s = (float*)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
  pair_t* order = (pair_t*)malloc(sizeof(pair_t) * (size_t)(n > 0 ? n : 1));
  if (!q || !s || !order) {
    free(q);
    free(s);
    free(order);
    return -1;
  }
  for (int32_t iq = 0; iq < nq; ++iq) {
    for (int32_t j = 0; j < d; ++j) q[j] = load_elem(Q, q_dtype, (int64_t)iq * d + j, round_bf16);
    score_one_query(X, x_dtype, n, d, q, normalize, round_bf16, threads, s);
    if (all_scores) memcpy(all_scores + (size_t)iq * (size_t)n, s, sizeof(float) * (size_t)n);
    for (int64_t i = 0; i < n; ++i) {
      order[i].score = s[i];
      order[i].slot = i;
    }
    qsort(order, (size_t)n, sizeof(pair_t), cmp_pair);
    for (int32_t r = 0; r < k; ++r) {
      size_t o = (size_t)iq * (size_t)k + (size_t)r;
      if (r < n) {
        int64_t slot = order[r].slot;
        if (out_ids) out_ids[o] = ids ? ids[slot] : slot;
        if (out_scores) out_scores[o] = order[r].score;
        if (out_slots) out_slots[o] = slot;
      } else {
        if (out_ids) out_ids[o] = -1;
        if (out_scores) out_scores[o] = -INFINITY;
        if (out_slots) out_slots[o] = -1;
      }
    }
  }
  free(q);
  free(s);
  free(order);
  return 0;
}

/*
 * Similarity-threshold filter on a search result (the hit test of semantic caching, paper
 * Sec. 2.2, and a similarity pre-filter before the utility threshold of Sec. 4.1): every
 * entry whose score is below min_score becomes (id -1, slot -1, score -inf); counts[q]
 * (optional) receives how many entries of query q remain.  Plain definition, entry by entry.
 */
void ic_oracle_apply_min_score(int64_t* out_ids, float* out_scores, int64_t* out_slots, int32_t nq, int32_t k,
                               float min_score, int32_t* counts) {
  for (int32_t iq = 0; iq < nq; ++iq) {
    int32_t kept = 0;
    for (int32_t r = 0; r < k; ++r) {
      size_t o = (size_t)iq * (size_t)k + (size_t)r;
      int present = out_scores[o] > -INFINITY || (out_ids && out_ids[o] != -1);
      if (present && out_scores[o] >= min_score) {
        ++kept;
      } else {
        if (out_ids) out_ids[o] = -1;
        if (out_slots) out_slots[o] = -1;
        out_scores[o] = -INFINITY;
      }
    }
    if (counts) counts[iq] = kept;
  }
}

/*
 * Top-1 similarity of cached entries to the OTHER cached entries (the request-similarity
 * study of paper Sec. 2.2: each request's best match among the other requests).
 * For every row i in [first, first+count): the row j != i with the largest fp32 dot product
 * (ties: lowest slot).  out_ids/out_slots/out_scores have `count` entries; with fewer than two
 * rows in the cache the answer is (-1, -1, -inf).  Plain double loop, no blocking.
 */
int ic_oracle_self_similarity(const void* X, int x_dtype, const int64_t* ids, int64_t n, int32_t d, int64_t first,
                              int64_t count, int threads, int64_t* out_ids, float* out_scores, int64_t* out_slots) {
  if (n < 0 || d <= 0 || first < 0 || count < 0 || first + count > n) return -1;
  if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
  for (int64_t r = 0; r < count; ++r) {
    const int64_t i = first + r;
    float best = -INFINITY;
    int64_t best_j = -1;
    for (int64_t j = 0; j < n; ++j) {
      if (j == i) continue;
      float acc = 0.0f;
      for (int32_t t = 0; t < d; ++t) acc += load_elem(X, x_dtype, i * (int64_t)d + t, 0) * load_elem(X, x_dtype, j * (int64_t)d + t, 0);
      if (best_j < 0 || acc > best) {
        best = acc;
        best_j = j;
      }
    }
    out_scores[r] = best;
    if (out_slots) out_slots[r] = best_j;
    if (out_ids) out_ids[r] = best_j < 0 ? -1 : (ids ? ids[best_j] : best_j);
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------
 * Two-level search (paper Sec. 4.1, "Two-Stage Scalable Example Selection": cached examples are
 * clustered offline into K groups with K-Means, K = sqrt(N) balancing the K centroid
 * comparisons against the N/K comparisons inside a cluster; a request is first matched to
 * centroids, then searched inside the closest clusters).
 *
 * The paper names the algorithm (K-Means) and nothing more, so this is textbook Lloyd iteration
 * under the retrieval metric: a row belongs to the centroid with the largest cosine (inner
 * product of unit vectors), a centroid is the mean of its rows scaled back to unit length
 * (spherical K-Means), stored as bf16 like every other embedding.  Steps in that order, no
 * blocking, no acceleration.
 * ------------------------------------------------------------------------------------------ */

/* Assignment step: assign[i] = the centroid with the largest fp32 dot product with row i (terms
 * added in index order), ties to the lower centroid index; best[i] (optional) = that product. */
int ic_oracle_kmeans_assign(const void* X, int x_dtype, int64_t n, int32_t d, const uint16_t* C, int32_t K,
                            int threads, int32_t* assign, float* best) {
  if (n < 0 || d <= 0 || K <= 0 || !C || !assign) return -1;
  if (threads < 1) threads = 1;
#pragma omp parallel for num_threads(threads) schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    float top = -INFINITY;
    int32_t top_c = -1;
    for (int32_t c = 0; c < K; ++c) {
      float acc = 0.0f;
      for (int32_t j = 0; j < d; ++j)
        acc += load_elem(X, x_dtype, i * (int64_t)d + j, 0) * ic_oracle_bf16_to_f32(C[(int64_t)c * d + j]);
      if (top_c < 0 || acc > top) {
        top = acc;
        top_c = c;
      }
    }
    assign[i] = top_c;
    if (best) best[i] = top;
  }
  return 0;
}

/* Update step: centroid c = (sum of its rows, fp64, rows in slot order) divided by that sum's
 * Euclidean norm, narrowed to fp32 and rounded to bf16 (nearest even).  A centroid without rows,
 * or whose rows sum to zero, keeps its previous value.  C_exact (optional, [K,d] doubles)
 * receives the unrounded unit vectors (previous value widened where kept); counts (optional)
 * the number of rows per centroid. */
int ic_oracle_kmeans_update(const void* X, int x_dtype, int64_t n, int32_t d, const int32_t* assign, int32_t K,
                            const uint16_t* C_prev, uint16_t* C_out, double* C_exact, int64_t* counts) {
  if (n < 0 || d <= 0 || K <= 0 || !assign || !C_prev || !C_out) return -1;
  double* sum = (double*)calloc((size_t)K * (size_t)d, sizeof(double));
  int64_t* cnt = (int64_t*)calloc((size_t)K, sizeof(int64_t));
  if (!sum || !cnt) {
    free(sum);
    free(cnt);
    return -1;
  }
  for (int64_t i = 0; i < n; ++i) {
    const int32_t c = assign[i];
    if (c < 0 || c >= K) {
      free(sum);
      free(cnt);
      return -1;
    }
    cnt[c] += 1;
    for (int32_t j = 0; j < d; ++j) sum[(int64_t)c * d + j] += (double)load_elem(X, x_dtype, i * (int64_t)d + j, 0);
  }
  for (int32_t c = 0; c < K; ++c) {
    double norm2 = 0.0;
    for (int32_t j = 0; j < d; ++j) norm2 += sum[(int64_t)c * d + j] * sum[(int64_t)c * d + j];
    const double norm = sqrt(norm2);
    for (int32_t j = 0; j < d; ++j) {
      const int64_t o = (int64_t)c * d + j;
      if (cnt[c] > 0 && norm > 0.0) {
        const double u = sum[o] / norm;
        C_out[o] = ic_oracle_f32_to_bf16((float)u);
        if (C_exact) C_exact[o] = u;
      } else {
        C_out[o] = C_prev[o];
        if (C_exact) C_exact[o] = (double)ic_oracle_bf16_to_f32(C_prev[o]);
      }
    }
    if (counts) counts[c] = cnt[c];
  }
  free(sum);
  free(cnt);
  return 0;
}

typedef struct {
  float score;
  int32_t c;
} cpair_t;

static int cmp_cpair(const void* a, const void* b) {
  const cpair_t* x = (const cpair_t*)a;
  const cpair_t* y = (const cpair_t*)b;
  if (x->score > y->score) return -1;
  if (x->score < y->score) return 1;
  return (x->c > y->c) - (x->c < y->c);
}

/*
 * Two-level retrieval.  Per query: (1) score all K centroids (fp32 dot product), order them by
 * score descending then index ascending, and probe the first min(nprobe, K); (2) score every row
 * that is assigned to a probed centroid, plus every row at slot >= n_indexed (rows added after the
 * clustering are always searched), and return the k best by score descending, slot ascending.
 *   assign [n_indexed]: centroid of each indexed row.
 *   probes_in: NULL, or [nq,nprobe] centroid indices to use instead of step (1) (-1 = none).
 *   out_probes (optional) [nq,nprobe]: the centroids probed, in order, -1 padded.
 *   centroid_scores (optional) [nq,K]; cand_scores (optional) [nq,n]: the score of every row that
 *   was searched, -inf for the others.
 */
int ic_oracle_search_clustered(const void* X, int x_dtype, const int64_t* ids, int64_t n, int32_t d, const void* Q,
                               int q_dtype, int32_t nq, int32_t k, const uint16_t* C, int32_t K, const int32_t* assign,
                               int64_t n_indexed, int32_t nprobe, const int64_t* probes_in, int threads,
                               int64_t* out_ids, float* out_scores, int64_t* out_slots, int64_t* out_probes,
                               float* centroid_scores, float* cand_scores) {
  if (n < 0 || d <= 0 || nq < 0 || k < 0 || K <= 0 || nprobe < 1 || n_indexed < 0 || n_indexed > n) return -1;
  if (!C || (n_indexed > 0 && !assign)) return -1;
  if (threads < 1) threads = 1;
  float* q = (float*)malloc(sizeof(float) * (size_t)d);
  float* s = (float*)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
  pair_t* order = (pair_t*)malloc(sizeof(pair_t) * (size_t)(n > 0 ? n : 1));
  cpair_t* cs = (cpair_t*)malloc(sizeof(cpair_t) * (size_t)K);
  unsigned char* probed = (unsigned char*)malloc((size_t)K);
  if (!q || !s || !order || !cs || !probed) {
    free(q); free(s); free(order); free(cs); free(probed);
    return -1;
  }
  for (int32_t iq = 0; iq < nq; ++iq) {
    for (int32_t j = 0; j < d; ++j) q[j] = load_elem(Q, q_dtype, (int64_t)iq * d + j, 0);
    /* step 1: the closest centroids */
    for (int32_t c = 0; c < K; ++c) {
      float acc = 0.0f;
      for (int32_t j = 0; j < d; ++j) acc += q[j] * ic_oracle_bf16_to_f32(C[(int64_t)c * d + j]);
      cs[c].score = acc;
      cs[c].c = c;
      if (centroid_scores) centroid_scores[(size_t)iq * (size_t)K + (size_t)c] = acc;
    }
    qsort(cs, (size_t)K, sizeof(cpair_t), cmp_cpair);
    memset(probed, 0, (size_t)K);
    for (int32_t p = 0; p < nprobe; ++p) {
      int64_t c = -1;
      if (probes_in) c = probes_in[(size_t)iq * (size_t)nprobe + (size_t)p];
      else if (p < K) c = cs[p].c;
      if (c >= K) { free(q); free(s); free(order); free(cs); free(probed); return -1; }
      if (c >= 0) probed[c] = 1;
      if (out_probes) out_probes[(size_t)iq * (size_t)nprobe + (size_t)p] = c;
    }
    /* step 2: exhaustive search inside the probed clusters and the rows added since */
    score_one_query(X, x_dtype, n, d, q, 0, 0, threads, s);
    int64_t m = 0;
    for (int64_t i = 0; i < n; ++i) {
      const int searched = (i >= n_indexed) || probed[assign[i]];
      if (cand_scores) cand_scores[(size_t)iq * (size_t)n + (size_t)i] = searched ? s[i] : -INFINITY;
      if (searched) {
        order[m].score = s[i];
        order[m].slot = i;
        ++m;
      }
    }
    qsort(order, (size_t)m, sizeof(pair_t), cmp_pair);
    for (int32_t r = 0; r < k; ++r) {
      size_t o = (size_t)iq * (size_t)k + (size_t)r;
      if (r < m) {
        int64_t slot = order[r].slot;
        if (out_ids) out_ids[o] = ids ? ids[slot] : slot;
        if (out_scores) out_scores[o] = order[r].score;
        if (out_slots) out_slots[o] = slot;
      } else {
        if (out_ids) out_ids[o] = -1;
        if (out_scores) out_scores[o] = -INFINITY;
        if (out_slots) out_slots[o] = -1;
      }
    }
  }
  free(q); free(s); free(order); free(cs); free(probed);
  return 0;
}
