/*
 * CPU oracle for IC-Cache stage-1 example retrieval.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product path links, imports or calls this file.  It shares no
 * code with the CUDA library.
 *
 * What it computes is the plain definition of the step, not an algorithm:
 *   - relevance of a cached example to a request = cosine similarity of their
 *     dense text embeddings (paper Sec. 4.1, "Example Selector", first paragraph;
 *     Sec. 2.2 similarity study: cosine, 1 = identical requests);
 *   - "prioritize examples with high similarity scores" (Sec. 4.1, two-stage
 *     selection paragraph) = return the k best-scoring cached examples;
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
 * library cross-check, closed-form statistics).
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
 * study of paper Sec. 2.2: "top-1 request similarities of each request to others").
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
