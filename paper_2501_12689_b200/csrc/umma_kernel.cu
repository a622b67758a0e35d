// Tensor-core path: scores = Q x X^T on tcgen05 with the partial top-k fused into the epilogue.
//
// Queries are the MMA M operand, cache rows the N operand (256 per accumulator), the embedding
// dimension is the K loop in 64-element (128-byte, swizzled) chunks.  With this orientation a
// tensor-memory lane of an accumulator holds the scores of one query against 256 consecutive
// cache rows, so the epilogue thread that owns the lane owns the query: its admission threshold
// stays in a register and a score costs a third of a compare unless it enters the list.
//
// Warp roles (192 threads, one CTA per SM):
//   warps 0-3  epilogue: tcgen05.ld the accumulator 64 columns at a time (one load in flight while
//              the previous one is filtered), reject whole groups by their maximum, push the rare
//              survivors into per-query queues and drain those into per-query heaps
//   warp 4     TMA producer
//   warp 5     MMA issuer (one thread) and tensor-memory owner
// Two 256-column accumulators alternate, so the epilogue of one row tile overlaps the MMAs
// of the next.  CTA (p, t) scores query tile t against row tiles p, p + P, p + 2P, ...
//
// Three instantiations:
//   <1, false>  128 queries per CTA; a ring stage holds a query chunk (16 KiB) and a row chunk (32 KiB)
//   <2, false>  CTA pairs: one 256 x 256 MMA per K step, each CTA stages its own 128 queries and
//               half of the row tile
//   <1, true>   at most 64 queries: M = 64, the whole query tile is loaded once and stays in
//               shared memory, ring stages hold 128 cache rows (16 KiB) and nothing else
//
// Threshold seeding inside the launch: every CTA first visits its first few tiles only for the
// maxima of four groups of 64 rows per query (the last of them with the accumulator held back)
// and publishes them; once the CTAs that score the same queries have all published (a bounded
// look, never a condition for progress), each epilogue thread folds all those maxima into bins of
// disjoint rows and takes a score that at least k bins reach as the floor of its query: k
// different rows score at least that much, so nothing below it can be in the top-k.  The tiles
// visited for their maxima only are scored at the end of the CTA's tile sequence.
#include <math.h>
#include <string.h>

#include "common.cuh"
#include "kernels.h"
#include "pipeline.cuh"

namespace icc {

constexpr int UM_THREADS = 192;
constexpr int UM_QT = 128;            // tensor-memory lanes = epilogue threads (queries per CTA unless resident)
constexpr int UM_RT = 256;            // cache rows per accumulator (MMA N, or two MMAs of N = 128)
constexpr int UM_KC = 64;             // elements per K chunk (128 bytes)
constexpr int UM_A_BYTES = UM_QT * UM_KC * 2;   // 16 KiB: 128 query rows of one K chunk
constexpr int UM_B_BYTES = UM_RT * UM_KC * 2;   // 32 KiB: 256 cache rows of one K chunk
constexpr int UM_QRES_CHUNK_BYTES = 64 * UM_KC * 2;   // 8 KiB: 64 resident query rows of one K chunk
// Bytes of one ring stage.  Streaming queries: the query chunk plus the CTA's share of the row
// chunk (all of it, or half with CTA pairs).  Resident queries: 128 cache rows.
template <int CG, bool QRES> __host__ __device__ constexpr int um_stage_bytes() {
  return QRES ? UM_B_BYTES / 2 : UM_A_BYTES + UM_B_BYTES / CG;
}
constexpr int UM_MAX_STAGES = 12;
constexpr int UM_TMEM_COLS = 512;
constexpr int UM_CHUNK = 64;          // accumulator columns per epilogue step
constexpr long long PACE_LIMIT_CYCLES = 100000;   // ~50 us: longest a CTA holds back for a slower sibling
constexpr uint32_t NAN_BITS = 0x7fc00000u;

struct UmmaSmemTail {
  uint64_t full[UM_MAX_STAGES];
  uint64_t empty[UM_MAX_STAGES];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t q_full;
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ float bits_f(uint32_t u) { return __uint_as_float(u); }
// Largest of eight consecutive values.
__device__ __forceinline__ float max8(const uint32_t* v) {
  return fmax3(fmax3(bits_f(v[0]), bits_f(v[1]), bits_f(v[2])), fmax3(bits_f(v[3]), bits_f(v[4]), bits_f(v[5])),
               fmaxf(bits_f(v[6]), bits_f(v[7])));
}
__device__ __forceinline__ float max8f(const float* g) {
  return fmax3(fmax3(g[0], g[1], g[2]), fmax3(g[3], g[4], g[5]), fmaxf(g[6], g[7]));
}

// Place `key` at the root of the 4-ary min-heap list[0 .. limit) (entry i at list[i * LW]; children of
// entry i are 4i+1 .. 4i+4) and sift it down; returns the new root, the smallest entry.  An all-empty
// list is a valid heap, so no fill phase exists.  Four children per level keep the chain of
// dependent shared-memory round trips short: log4(k) levels.
template <int LW>
__device__ __forceinline__ uint64_t heap_replace_root(uint64_t* list, uint64_t key, int limit) {
  int pos = 0;
  uint64_t root = key;
  while (true) {
    const int c0 = 4 * pos + 1;
    if (c0 >= limit) break;
    const uint64_t v0 = list[c0 * LW];
    const uint64_t v1 = (c0 + 1 < limit) ? list[(c0 + 1) * LW] : ~0ull;
    const uint64_t v2 = (c0 + 2 < limit) ? list[(c0 + 2) * LW] : ~0ull;
    const uint64_t v3 = (c0 + 3 < limit) ? list[(c0 + 3) * LW] : ~0ull;
    const bool b01 = v1 < v0, b23 = v3 < v2;
    const uint64_t m01 = b01 ? v1 : v0, m23 = b23 ? v3 : v2;
    const int i01 = b01 ? c0 + 1 : c0, i23 = b23 ? c0 + 3 : c0 + 2;
    const bool hi = m23 < m01;
    const uint64_t cv = hi ? m23 : m01;
    if (cv >= key) break;
    list[pos * LW] = cv;
    if (pos == 0) root = cv;
    pos = hi ? i23 : i01;
  }
  list[pos * LW] = key;
  return root;
}

// Admission state of one query, kept in registers by its epilogue thread.
struct Admission {
  uint64_t thr_key;    // candidates must beat this key: the heap's root once it is full, else the floor
  float thr_score;     // its score: the cheap first test
};

// Empty a thread's queue of `cnt` candidates ((score bits << 32) | slot, entry i at queue[i * LW])
// into its heap.  Deliberately not inlined: it is called from many places in the filter, runs
// rarely, and its code would otherwise be copied into each of them (the filter is meant to stay in
// the instruction cache).  No warp-wide operation inside: lanes run it with different counts.
template <int LW>
__device__ __noinline__ Admission drain_queue(Admission a, uint64_t thr_floor, uint64_t* list, const uint64_t* queue,
                                              int cnt, int k) {
  for (int i = 0; i < cnt; ++i) {
    const uint64_t raw = queue[i * LW];
    const uint64_t key = make_key(__uint_as_float((uint32_t)(raw >> 32)), (uint32_t)raw);
    if (key > a.thr_key) {
      const uint64_t root = heap_replace_root<LW>(list, key, k);
      a.thr_key = root > thr_floor ? root : thr_floor;
      a.thr_score = (a.thr_key == KEY_EMPTY) ? -INFINITY : key_score(a.thr_key);
    }
  }
  return a;
}

// What a thread carries through the filter: its admission state and the fill of its queue.
struct Filter {
  Admission a;
  int cnt;
};

// One group of eight accumulator columns (cache rows col_first .. col_first+7) in which some lane of
// the warp has a passing score: every lane pushes its passing ones.  Called by all 32 lanes together
// (it votes).  Before the pushes the queues are drained, all lanes at once, unless every lane still
// has room for eight more entries; queues shorter than a group (very long lists leave little shared
// memory) are served one column at a time.  Not inlined, like drain_queue: the filter calls it from
// sixteen places and runs it rarely.
template <int LW>
__device__ __noinline__ Filter admit_group(Filter f, uint64_t thr_floor, uint64_t* list, uint64_t* queue, int qcap, int k,
                                           uint32_t col_first, uint32_t v0, uint32_t v1, uint32_t v2, uint32_t v3,
                                           uint32_t v4, uint32_t v5, uint32_t v6, uint32_t v7) {
  const uint32_t v[8] = {v0, v1, v2, v3, v4, v5, v6, v7};
  if (qcap >= 8) {
    if (__any_sync(FULL_MASK, f.cnt + 8 > qcap)) {
      f.a = drain_queue<LW>(f.a, thr_floor, list, queue, f.cnt, k);
      f.cnt = 0;
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      if (__uint_as_float(v[c]) >= f.a.thr_score) {
        queue[f.cnt * LW] = ((uint64_t)v[c] << 32) | (uint64_t)(col_first + c);
        ++f.cnt;
      }
    }
  } else {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      if (__any_sync(FULL_MASK, f.cnt >= qcap)) {
        f.a = drain_queue<LW>(f.a, thr_floor, list, queue, f.cnt, k);
        f.cnt = 0;
      }
      if (__uint_as_float(v[c]) >= f.a.thr_score) {
        queue[f.cnt * LW] = ((uint64_t)v[c] << 32) | (uint64_t)(col_first + c);
        ++f.cnt;
      }
    }
  }
  return f;
}

template <int CG, bool QRES>
__global__ void __launch_bounds__(UM_THREADS, 1)
umma_score_topk_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_slab,
                       int64_t n, int64_t tile_begin, int64_t tile_end, int dim, int nq, int k, int n_query_tiles,
                       int n_part, int n_stages, int qcap, const uint64_t* __restrict__ thr_floor_in,
                       uint64_t* __restrict__ partials, unsigned long long* pace, unsigned epoch, int pace_window,
                       float* seed_maxima, unsigned* seed_flags, int seed_t0, int seed_look_cycles, int* dev_status) {
  static_assert(!(QRES && CG == 2), "resident queries run on single CTAs");
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int STAGE_BYTES = um_stage_bytes<CG, QRES>();
  constexpr int LW = QRES ? 16 : 32;       // list owners per epilogue warp (tensor-memory lanes that hold queries)
  constexpr int QPC = QRES ? 64 : UM_QT;   // queries per CTA
  const int n_kc = (dim + UM_KC - 1) / UM_KC;
  unsigned char* qres = smem;                                                        // QRES: n_kc chunks of 8 KiB
  unsigned char* ring = smem + (QRES ? (size_t)n_kc * UM_QRES_CHUNK_BYTES : 0);      // n_stages * STAGE_BYTES
  uint64_t* lists = reinterpret_cast<uint64_t*>(ring + (size_t)n_stages * STAGE_BYTES);  // [4 warps][k][LW]
  uint64_t* queues = lists + (size_t)4 * LW * k;                                     // [4 warps][qcap][LW]
  UmmaSmemTail* tail = reinterpret_cast<UmmaSmemTail*>(queues + (size_t)4 * LW * qcap);
  volatile int* abort_flag = &tail->abort_flag;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // CG == 1: CTA b scores query tile b % nqt against partition b / nqt.  CG == 2: CTAs 2c and
  // 2c+1 form a pair that scores query tiles 2*(c % (nqt/2)) + rank against partition
  // c / (nqt/2); rank 0 issues the MMAs for both.
  const uint32_t rank = (CG == 2) ? cluster_ctarank() : 0u;
  const int unit = (CG == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int units_per_part = n_query_tiles / CG;
  const int qt = (unit % units_per_part) * CG + (int)rank;   // query tile of this CTA
  const int part = unit / units_per_part;                    // row partition of this CTA
  // This launch scores row tiles [tile_begin, tile_end); CTA (part, qt) takes every n_part-th:
  // n_my tiles.  With seeding inside the launch the first n_pre of them are first read for their
  // group maxima only and come round again, to be scored, at the end of the sequence.
  const int64_t span = tile_end - tile_begin - part;
  const int64_t n_my = span > 0 ? (span + n_part - 1) / n_part : 0;
  const bool self_seed = seed_maxima != nullptr && thr_floor_in == nullptr && n_my >= seed_t0;
  const int n_pre = self_seed ? seed_t0 - 1 : 0;
  const int64_t n_seq = n_my > 0 ? n_my + n_pre : 0;
  auto tile_of = [&](int64_t sq) -> int64_t { return tile_begin + part + (int64_t)n_part * (sq < n_my ? sq : sq - n_my); };

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&tail->full[s], CG);       // one arrive.expect_tx per producing CTA
      mbar_init(&tail->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tail->acc_full[b], 1);
      mbar_init(&tail->acc_empty[b], 4 * CG);  // one arrival per epilogue warp of every CTA
    }
    mbar_init(&tail->q_full, 1);
    mbar_init(&tail->drain, 1);
    tail->abort_flag = 0;
    mbar_fence_init();
  }
  for (int i = tid; i < 4 * LW * k; i += UM_THREADS) lists[i] = KEY_EMPTY;
  if (warp == 4 && lane == 0) {
    prefetch_tmap(&tmap_q);
    prefetch_tmap(&tmap_slab);
  }
  if (warp == 5) {
    if (CG == 2) tmem_alloc_pair(&tail->tmem_base, UM_TMEM_COLS);
    else tmem_alloc(&tail->tmem_base, UM_TMEM_COLS);
  }
  grid_dep_launch_dependents();
  grid_dep_wait();   // queries, thresholds and new rows come from earlier kernels in the stream
  tc_fence_before_sync();
  __syncthreads();
  if (CG == 2) cluster_sync_all();   // the peer's barriers are initialised before anyone signals them
  tc_fence_after_sync();
  // barriers the pair shares live in the rank-0 CTA
  const uint32_t lead_full0 = (CG == 2) ? mapa_shared(smem_u32(&tail->full[0]), 0) : smem_u32(&tail->full[0]);
  const uint32_t lead_acc_empty0 = (CG == 2) ? mapa_shared(smem_u32(&tail->acc_empty[0]), 0) : smem_u32(&tail->acc_empty[0]);
  const uint32_t tmem_base = tail->tmem_base;

  if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int64_t it = 0;
      int s = 0;          // ring stage and the parity of its current use: plain counters, because a
      uint32_t ph = 0;    // 64-bit division per K chunk would cost this single thread more than the chunk's MMAs
      bool ok = true;
      if (QRES) {
        // the whole query tile, once: n_kc boxes of 64 rows x 64 elements
        mbar_arrive_expect_tx(&tail->q_full, (uint32_t)(n_kc * UM_QRES_CHUNK_BYTES));
        for (int kc = 0; kc < n_kc; ++kc)
          tma_load_2d(qres + (size_t)kc * UM_QRES_CHUNK_BYTES, &tmap_q, kc * UM_KC, qt * QPC, &tail->q_full);
      }
      // Pacing.  The CTAs (or pairs) that score different query tiles against the same
      // partition read the same row tiles; the tile comes from HBM once only while they stay
      // within an L2-sized window of each other.  They normally do by themselves (the ones behind
      // find the tiles in L2 and catch up), so this is insurance against data-dependent drift and
      // is kept cheap: only every PACE_EVERY-th tile a CTA publishes how many tiles it has started
      // and looks at the others (a round trip to L2 that stalls this thread while the ring
      // drains); one that is more than pace_window tiles ahead of the slowest word holds its
      // loads for a bounded time.  A bandwidth hint only: when the bound runs out it goes on.
      const bool paced = (pace != nullptr) && units_per_part > 1 && rank == 0;
      volatile unsigned long long* pace_row = paced ? pace + (size_t)part * units_per_part : nullptr;
      const int my_unit = unit % units_per_part;
      uint32_t ordinal = 0;
      constexpr int SUB = QRES ? 2 : 1;    // ring stages per K chunk of a row tile (resident: two halves of 128 rows)
      for (int64_t sq = 0; sq < n_seq && ok; ++sq, ++ordinal) {
        const int64_t tile = tile_of(sq);
        const bool look = paced && (ordinal % PACE_EVERY) == 0;
        if (look) pace_row[my_unit] = ((unsigned long long)epoch << 32) | ordinal;
        for (int sub = 0; sub < SUB && ok; ++sub) {
          for (int kc = 0; kc < n_kc; ++kc, ++it) {
            ok = mbar_wait(&tail->empty[s], ph ^ 1u, abort_flag);
            if (!ok) break;
            if (look && kc == 0 && sub == 0) {
              const long long t0 = clock64();
              while (true) {
                // all progress words are requested before the first is looked at (one round trip to
                // L2, not one per sibling); there are at most eight siblings
                unsigned long long w[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) w[u] = pace_row[u < units_per_part ? u : my_unit];
                uint32_t slowest = ordinal;
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                  const uint32_t o = ((uint32_t)(w[u] >> 32) == epoch) ? (uint32_t)w[u] : 0u;   // not started yet
                  slowest = o < slowest ? o : slowest;
                }
                if (ordinal - slowest <= (uint32_t)pace_window || clock64() - t0 > PACE_LIMIT_CYCLES) break;
                __nanosleep(200);
              }
            }
            unsigned char* a_dst = ring + (size_t)s * STAGE_BYTES;
            if (QRES) {
              mbar_arrive_expect_tx(&tail->full[s], STAGE_BYTES);
              tma_load_2d(a_dst, &tmap_slab, kc * UM_KC, (int)(tile * UM_RT) + sub * (UM_RT / 2), &tail->full[s]);
            } else if (CG == 2) {
              const uint32_t full = lead_full0 + (uint32_t)(s * 8);
              mbar_arrive_expect_tx_cluster(full, STAGE_BYTES);
              tma_load_2d_pair(a_dst, &tmap_q, kc * UM_KC, qt * UM_QT, full);
              tma_load_2d_pair(a_dst + UM_A_BYTES, &tmap_slab, kc * UM_KC, (int)(tile * UM_RT) + (int)rank * (UM_RT / 2), full);
            } else {
              mbar_arrive_expect_tx(&tail->full[s], STAGE_BYTES);
              tma_load_2d(a_dst, &tmap_q, kc * UM_KC, qt * UM_QT, &tail->full[s]);
              tma_load_2d(a_dst + UM_A_BYTES, &tmap_slab, kc * UM_KC, (int)(tile * UM_RT), &tail->full[s]);
            }
            if (++s == n_stages) {
              s = 0;
              ph ^= 1u;
            }
          }
        }
      }
      if (!ok) {
        report_status(dev_status, DEV_TIMEOUT_MBAR);
        // loads already issued still write this CTA's shared memory: wait for them (bounded)
        for (int64_t j = (it > n_stages ? it - n_stages : 0); j < it && rank == 0; ++j) {
          const int sj = (int)(j % n_stages);   // (failure path only)
          const long long t0 = clock64();
          while (!mbar_try_wait(&tail->full[sj], (uint32_t)((j / n_stages) & 1)) &&
                 clock64() - t0 < WAIT_LIMIT_CYCLES) {
          }
        }
      }
      if (QRES) {   // the query tile's loads, too, have landed before the CTA leaves
        const long long t0 = clock64();
        while (!mbar_try_wait(&tail->q_full, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      // streaming: one M x 256 MMA per 16 elements of K; resident queries: M = 64 and two
      // accumulator halves of 128 columns, each fed by its own run of ring stages
      constexpr uint32_t idesc = QRES ? umma_idesc_bf16_f32(64, UM_RT / 2) : umma_idesc_bf16_f32(UM_QT * CG, UM_RT);
      constexpr int SUB = QRES ? 2 : 1;
      int s = 0;          // ring stage and parity as plain counters (see the producer)
      uint32_t ph = 0;
      int64_t lt = 0;
      bool ok = true;
      const uint32_t ring_addr = smem_u32(ring);
      const uint32_t qres_addr = smem_u32(qres);
      if (QRES) {
        ok = mbar_wait(&tail->q_full, 0, abort_flag);
        tc_fence_after_sync();
      }
      for (; lt < n_seq && ok; ++lt) {
        const int buf = (int)(lt & 1);
        const uint32_t bph = (uint32_t)((lt >> 1) & 1);
        ok = mbar_wait(&tail->acc_empty[buf], bph ^ 1u, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        for (int sub = 0; sub < SUB && ok; ++sub) {
          const uint32_t d_tmem = tmem_base + (uint32_t)(buf * UM_RT + sub * (UM_RT / 2));
          for (int kc = 0; kc < n_kc; ++kc) {
            ok = mbar_wait(&tail->full[s], ph, abort_flag);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t st_addr = ring_addr + (uint32_t)(s * STAGE_BYTES);
            const uint64_t da = umma_desc_k_major_sw128(QRES ? qres_addr + (uint32_t)(kc * UM_QRES_CHUNK_BYTES) : st_addr);
            const uint64_t db = umma_desc_k_major_sw128(QRES ? st_addr : st_addr + UM_A_BYTES);
#pragma unroll
            for (int kk = 0; kk < UM_KC / 16; ++kk) {
              // 16 bf16 = 32 bytes further along K inside the swizzled 128-byte row
              if (CG == 2) umma_bf16_pair(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (kc | kk) != 0 ? 1u : 0u);
              else umma_bf16(d_tmem, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (kc | kk) != 0 ? 1u : 0u);
            }
            // stage reusable (in both CTAs of a pair) once these MMAs have read it
            if (CG == 2) umma_commit_pair_both(&tail->empty[s]);
            else umma_commit(&tail->empty[s]);
            if (++s == n_stages) {
              s = 0;
              ph ^= 1u;
            }
          }
        }
        if (ok) {
          if (CG == 2) umma_commit_pair_both(&tail->acc_full[buf]);
          else umma_commit(&tail->acc_full[buf]);
        }
      }
      // make sure nothing issued is still running before tensor memory is released
      if (CG == 2) umma_commit_pair(&tail->drain);
      else umma_commit(&tail->drain);
      {
        const long long t0 = clock64();
        while (!mbar_try_wait(&tail->drain, 0) && clock64() - t0 < WAIT_LIMIT_CYCLES) {
        }
      }
      if (!ok) report_status(dev_status, DEV_TIMEOUT_MBAR);
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 0-3)
    // A thread owns one tensor-memory lane, i.e. one query.  Streaming: thread t owns query
    // qt*128 + t.  Resident (M = 64): an accumulator keeps query 16w + l in lane 32w + l, l < 16,
    // so the first 16 threads of warp w own queries and the others own nothing.
    // The k best candidates of a query live in a private 4-ary min-heap in shared memory, stored
    // transposed ([k][LW] per warp) so that the lanes of a warp touch consecutive 8-byte words.
    // The admission threshold (root of the heap, or the seeded floor) stays in registers.
    // A score that passes the threshold is only appended to the thread's small queue; the queues
    // are drained with all lanes working on their own heap at the same time.
    const bool owns = lane < LW;
    const int q_local = QRES ? warp * 16 + lane : tid;
    const int q = qt * QPC + q_local;
    const bool real = owns && q < nq;
    uint64_t* warp_lists = lists + (size_t)(warp * LW) * k;
    uint64_t* my_list = warp_lists + (lane & (LW - 1));                              // entry i at my_list[i * LW]
    uint64_t* my_queue = queues + (size_t)(warp * LW) * qcap + (lane & (LW - 1));    // entry i at my_queue[i * LW]
    // A seeding pass over a sample of the rows may have established that k entries with keys
    // >= thr_floor exist: nothing at or below that key can be in the final top-k.
    uint64_t thr_floor = (real && thr_floor_in) ? thr_floor_in[q] : KEY_EMPTY;
    uint64_t thr_key = thr_floor;
    float thr_score = !real ? bits_f(NAN_BITS)                          // NaN never admits
                            : (thr_floor == KEY_EMPTY ? -INFINITY : key_score(thr_floor));
    int cnt = 0;
    auto drain = [&]() {
      const Admission a = drain_queue<LW>(Admission{thr_key, thr_score}, thr_floor, my_list, my_queue, cnt, k);
      thr_key = a.thr_key;
      thr_score = a.thr_score;
      cnt = 0;
    };
    // Filter 64 accumulator columns (cache rows col0 .. col0+63) held in registers.  Common case:
    // the maxima of the eight groups of eight and their maximum (36 three-input max
    // instructions) show that no lane has a passing column, and one vote ends it.  Otherwise the
    // groups in which any lane has one are handed, under warp-uniform branches (no divergence),
    // to admit_group.
    auto process = [&](uint32_t (&v)[UM_CHUNK], int64_t col0) {
      if (col0 >= n) return;                          // (warp-uniform) rows past the end score 0: ignore
      if (col0 + UM_CHUNK > n) {                      // ragged last tile: columns past n never admit
#pragma unroll
        for (int c = 0; c < UM_CHUNK; ++c)
          if (col0 + c >= n) v[c] = NAN_BITS;
      }
      float g[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) g[j] = max8(&v[8 * j]);
      const float m = max8f(g);
      if (!__any_sync(FULL_MASK, m >= thr_score)) return;
      uint32_t gm = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) gm |= (g[j] >= thr_score) ? (1u << j) : 0u;
      const uint32_t um = __reduce_or_sync(FULL_MASK, gm);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if ((um >> j) & 1u) {                         // warp-uniform
          const Filter f = admit_group<LW>(Filter{Admission{thr_key, thr_score}, cnt}, thr_floor, my_list, my_queue, qcap, k,
                                           (uint32_t)(col0 + 8 * j), v[8 * j], v[8 * j + 1], v[8 * j + 2], v[8 * j + 3],
                                           v[8 * j + 4], v[8 * j + 5], v[8 * j + 6], v[8 * j + 7]);
          thr_key = f.a.thr_key;
          thr_score = f.a.thr_score;
          cnt = f.cnt;
        }
      }
    };

    int64_t lt = 0;
    bool ok = true;
    for (; lt < n_seq; ++lt) {
      const int64_t tile = tile_of(lt);
      ICC_CHECK(tile >= tile_begin && tile < tile_end && cnt >= 0 && cnt <= qcap, dev_status);
      const int buf = (int)(lt & 1);
      const uint32_t bph = (uint32_t)((lt >> 1) & 1);
      ok = mbar_wait(&tail->acc_full[buf], bph, abort_flag);
      ok = __all_sync(FULL_MASK, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t t_addr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * UM_RT);
      const int64_t row0 = tile * UM_RT;
      float4* seed_base = self_seed ? reinterpret_cast<float4*>(seed_maxima) + (size_t)qt * n_part * seed_t0 * UM_QT : nullptr;
      if (lt < n_pre) {
        // Maxima-only visit of one of the CTA's first tiles: per query the best score of each of
        // its four groups of 64 rows goes to global memory and the accumulator is handed back.
        // The tile is scored for real at the end of the sequence, when the thresholds are tight.
        float mx[4];
#pragma unroll
        for (int cp = 0; cp < 4; ++cp) {
          uint32_t v[UM_CHUNK];
          tmem_ld_32x64(t_addr + (uint32_t)(cp * UM_CHUNK), v);
          tmem_ld_wait_for(v);
          float g[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) g[j] = max8(&v[8 * j]);
          mx[cp] = max8f(g);
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(lead_acc_empty0 + (uint32_t)(buf * 8));
        if (owns) seed_base[((size_t)part * seed_t0 + lt) * UM_QT + q_local] = make_float4(mx[0], mx[1], mx[2], mx[3]);
        continue;
      }
      if (lt == n_pre && thr_floor_in == nullptr && row0 + UM_RT <= n && (self_seed || k <= 32)) {
        // First tile that is scored, in a launch that was given no floors: read the accumulator once
        // just for the maxima of its 32 groups of 8 columns (and of its 4 groups of 64), before any
        // list exists.
        float g32[32], mx[4];
#pragma unroll
        for (int cp = 0; cp < 4; ++cp) {
          uint32_t v[UM_CHUNK];
          tmem_ld_32x64(t_addr + (uint32_t)(cp * UM_CHUNK), v);
          tmem_ld_wait_for(v);
#pragma unroll
          for (int j = 0; j < 8; ++j) g32[8 * cp + j] = max8(&v[8 * j]);
          mx[cp] = max8f(&g32[8 * cp]);
        }
        bool have_floor = false, sort_g32 = false;
        if (self_seed) {
          // Seeding across the launch.  Publish this tile's four maxima per query (those of the
          // maxima-only tiles are there already); then look, for a bounded time, whether every CTA
          // that scores the same queries against another partition has published too.  The
          // accumulator stays unread meanwhile (the MMA issuer fills the other one and the ring,
          // then waits), so what this costs is the part of the look and of the selection below that
          // exceeds about one tile's time.  If the siblings do not show up in time the tile is
          // scored with the local floor further down instead.
          if (owns) seed_base[((size_t)part * seed_t0 + n_pre) * UM_QT + q_local] = make_float4(mx[0], mx[1], mx[2], mx[3]);
          // one flag per epilogue warp: a thread only ever reads what the same warp of a sibling
          // CTA wrote (its own query's entries), so no CTA-wide step is needed
          __threadfence();
          __syncwarp();
          if (lane == 0) st_release_gpu(seed_flags + (size_t)(qt * n_part + part) * 4 + warp, epoch);
          const unsigned* fl = seed_flags + (size_t)qt * n_part * 4 + warp;
          const long long t0 = clock64();
          bool complete;
          while (true) {
            bool all = true;
            for (int p = lane; p < n_part; p += 32) all = all && (ld_acquire_gpu(fl + p * 4) == epoch);
            complete = __all_sync(FULL_MASK, all);
            if (complete || __any_sync(FULL_MASK, clock64() - t0 > (long long)seed_look_cycles)) break;
            __nanosleep(256);
          }
          const int n_ent = n_part * seed_t0;          // float4 entries per query: 4 * n_ent group maxima
          const float4* mine = seed_base + (owns ? q_local : 0);
          if (complete && k <= 16 && n_ent * 4 >= 32) {
            // Few results: fold the maxima into 32 bins by maximum (bin = value number mod 32:
            // straight-line code on registers, no lane ever waits for another) and let the sorting
            // network below take the k-th largest bin.  Bins are disjoint sets of rows, so k
            // different rows score at least that much; with 32 bins and k <= 16 the floor is within
            // a few tens of percent (in tail probability) of the k-th largest of all maxima.
#pragma unroll
            for (int i = 0; i < 32; ++i) g32[i] = -INFINITY;
            for (int e0 = 0; e0 < n_ent; e0 += 8) {
              float4 gv[8];
#pragma unroll
              for (int u = 0; u < 8; ++u)
                gv[u] = (e0 + u < n_ent) ? __ldcg(mine + (size_t)(e0 + u) * UM_QT)
                                         : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll
              for (int u = 0; u < 8; ++u) {
                g32[4 * u] = fmaxf(g32[4 * u], gv[u].x);
                g32[4 * u + 1] = fmaxf(g32[4 * u + 1], gv[u].y);
                g32[4 * u + 2] = fmaxf(g32[4 * u + 2], gv[u].z);
                g32[4 * u + 3] = fmaxf(g32[4 * u + 3], gv[u].w);
              }
            }
            sort_g32 = true;
          } else if (complete && n_ent * 4 >= k) {
            // Longer lists: fold the maxima into up to 2k bins kept in the thread's (still unused)
            // list space, then bisect on the score for a value that at least k bins reach.  The same
            // instructions in every lane, nothing data-dependent but selects; the result is a valid
            // floor at every step (the lower end always has k bins at or above it) and after ten
            // halvings of the bins' range it is as good as their exact k-th largest.
            // Two bins share one 8-byte list entry and are updated together.  With at least as many
            // entries as bins an entry goes in as the maximum of its four values (the rows covered
            // stay the same, a quarter of the updates); with fewer, as two maxima of two, or as is.
            const int per_entry = (n_ent >= 2 * k) ? 1 : (2 * n_ent >= 2 * k ? 2 : 4);
            const int n_pairs = min(2 * k, n_ent * per_entry) >> 1;      // pairs of bins, at least k / 2 ... k
            float2* bins = reinterpret_cast<float2*>(my_list);           // pair b at bins[b * LW]
            if (owns)
              for (int b2 = 0; b2 < n_pairs; ++b2) bins[b2 * LW] = make_float2(-INFINITY, -INFINITY);
            int cur = 0;
            float carry = -INFINITY;    // per_entry == 1: the first value of a pair waits here for the second
            for (int e0 = 0; e0 < n_ent; e0 += 16) {
              float4 gv[16];   // sixteen loads in flight: the round trips to L2 are what this loop waits for
#pragma unroll
              for (int u = 0; u < 16; ++u)
                gv[u] = (e0 + u < n_ent) ? __ldcg(mine + (size_t)(e0 + u) * UM_QT)
                                         : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll
              for (int u = 0; u < 16; ++u) {
                if (e0 + u < n_ent) {                 // (warp-uniform, like everything that steers this loop)
                  const float m01 = fmaxf(gv[u].x, gv[u].y), m23 = fmaxf(gv[u].z, gv[u].w);
                  if (per_entry == 1) {
                    const float mval = fmaxf(m01, m23);
                    if (((e0 + u) & 1) == 0) {
                      carry = mval;
                    } else {
                      if (owns) {
                        const float2 old = bins[cur * LW];
                        bins[cur * LW] = make_float2(fmaxf(old.x, carry), fmaxf(old.y, mval));
                      }
                      cur = (cur + 1 == n_pairs) ? 0 : cur + 1;
                    }
                  } else {
                    const float2 first = per_entry == 2 ? make_float2(m01, m23) : make_float2(gv[u].x, gv[u].y);
                    if (owns) {
                      const float2 old = bins[cur * LW];
                      bins[cur * LW] = make_float2(fmaxf(old.x, first.x), fmaxf(old.y, first.y));
                    }
                    cur = (cur + 1 == n_pairs) ? 0 : cur + 1;
                    if (per_entry == 4) {
                      if (owns) {
                        const float2 old = bins[cur * LW];
                        bins[cur * LW] = make_float2(fmaxf(old.x, gv[u].z), fmaxf(old.y, gv[u].w));
                      }
                      cur = (cur + 1 == n_pairs) ? 0 : cur + 1;
                    }
                  }
                }
              }
            }
            float lo = INFINITY, hi = -INFINITY;
            for (int b2 = 0; b2 < n_pairs; ++b2) {
              const float2 x = owns ? bins[b2 * LW] : make_float2(0.0f, 0.0f);
              lo = fminf(lo, fminf(x.x, x.y));
              hi = fmaxf(hi, fmaxf(x.x, x.y));
            }
            for (int round = 0; round < 10; ++round) {
              const float mid = 0.5f * (lo + hi);
              int reach = 0;
              for (int b2 = 0; b2 < n_pairs; ++b2) {
                const float2 x = owns ? bins[b2 * LW] : make_float2(0.0f, 0.0f);
                reach += (x.x >= mid ? 1 : 0) + (x.y >= mid ? 1 : 0);
              }
              lo = (reach >= k) ? mid : lo;
              hi = (reach >= k) ? hi : mid;
            }
            if (owns)
              for (int i = 0; i < k; ++i) my_list[i * LW] = KEY_EMPTY;
            if (real && 2 * n_pairs >= k && lo > -INFINITY && lo == lo) {   // (fewer than k bins: no floor)
              // admit every key whose score is >= the floor: the smallest such key has slot word 0
              thr_floor = ((uint64_t)score_to_ord(lo) << 32) - 1;
              thr_key = thr_floor;
              thr_score = lo;
            }
            have_floor = true;
          }
        }
        if (sort_g32 || (!have_floor && k <= 32)) {
          // The k-th largest of 32 maxima of disjoint groups of rows: the bins above, or else this
          // tile's own 32 groups of 8 columns (a local floor: k different columns score at least
          // that much, so only a few percent of the columns pass instead of every column passing
          // an empty list).  Bitonic sorting network, descending, on registers.
#pragma unroll
          for (int ls = 1; ls <= 5; ++ls) {
#pragma unroll
            for (int lj = 4; lj >= 0; --lj) {
              if (lj < ls) {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                  const int j = i ^ (1 << lj);
                  if (j > i) {
                    const bool desc = (i & (1 << ls)) == 0;
                    const float hi = fmaxf(g32[i], g32[j]), lo = fminf(g32[i], g32[j]);
                    g32[i] = desc ? hi : lo;
                    g32[j] = desc ? lo : hi;
                  }
                }
              }
            }
          }
          // sorted descending: the k-th entry is the largest of the entries k-1 .. 31
          float tau = -INFINITY;
#pragma unroll
          for (int i = 0; i < 32; ++i) tau = fmaxf(tau, i >= k - 1 ? g32[i] : -INFINITY);
          if (real && tau == tau && tau > -INFINITY) {
            thr_floor = ((uint64_t)score_to_ord(tau) << 32) - 1;
            thr_key = thr_floor;
            thr_score = tau;
          }
        }
      }
      // Tensor-memory loads take several hundred cycles while MMAs are running: the next 64
      // columns are requested before the current 64 are filtered.
      uint32_t va[UM_CHUNK], vb[UM_CHUNK];
      tmem_ld_32x64(t_addr, va);
#pragma unroll 1
      for (int h = 0; h < 2; ++h) {
        tmem_ld_wait_for(va);
        tmem_ld_32x64(t_addr + (uint32_t)(h * 128 + 64), vb);
        process(va, row0 + h * 128);
        tmem_ld_wait_for(vb);
        if (h == 0) {
          tmem_ld_32x64(t_addr + 128u, va);
        } else {
          // the accumulator has been read completely: hand it back to the MMA issuer
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(lead_acc_empty0 + (uint32_t)(buf * 8));
        }
        process(vb, row0 + h * 128 + 64);
      }
    }
    if (!ok && lane == 0) report_status(dev_status, DEV_TIMEOUT_MBAR);
    drain();
    if (owns) {
      // sort the private list descending, lanes in parallel: heapsort in place (the smallest
      // entry goes to the end of the shrinking heap)
      for (int end = k - 1; end > 0; --end) {
        const uint64_t smallest = my_list[0];
        const uint64_t moved = my_list[end * LW];
        my_list[end * LW] = smallest;
        heap_replace_root<LW>(my_list, moved, end);
      }
    }
    __syncwarp();
    // transpose out: the partial lists of this warp's queries are contiguous in global memory
    const int q_first = qt * QPC + warp * LW;
    const int q_live = min(LW, nq - q_first);
    if (q_live > 0) {
      uint64_t* dst = partials + ((size_t)part * nq + q_first) * k;
      ICC_CHECK(part < n_part && q_first + q_live <= nq, dev_status);
      for (int i = lane; i < q_live * k; i += 32) {
        const int ql = i / k, e = i - ql * k;
        const uint64_t key = warp_lists[e * LW + ql];
        // a list holds real rows only, best first
        ICC_CHECK(key == KEY_EMPTY || (int64_t)key_slot(key) < n, dev_status);
        ICC_CHECK(e == 0 || key <= warp_lists[(e - 1) * LW + ql], dev_status);
        dst[i] = key;
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (CG == 2) cluster_sync_all();   // neither CTA leaves while the other may still signal it
  if (warp == 5) {
    tc_fence_after_sync();
    if (CG == 2) tmem_dealloc_pair(tmem_base, UM_TMEM_COLS);
    else tmem_dealloc(tmem_base, UM_TMEM_COLS);
  }
}

cudaError_t umma_configure(int smem_optin) {
  cudaError_t e = cudaFuncSetAttribute(umma_score_topk_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(umma_score_topk_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(umma_score_topk_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  return e;
}

size_t umma_smem_bytes(int cta_group, bool q_resident, int dim, int k, int queue_cap, int n_stages) {
  const int n_kc = (dim + UM_KC - 1) / UM_KC;
  const int stage = q_resident ? um_stage_bytes<1, true>() : (cta_group == 2 ? um_stage_bytes<2, false>() : um_stage_bytes<1, false>());
  const int owners = q_resident ? 64 : UM_QT;
  return 1024 + (q_resident ? (size_t)n_kc * UM_QRES_CHUNK_BYTES : 0) + (size_t)n_stages * stage +
         (size_t)owners * (k + queue_cap) * 8 + sizeof(UmmaSmemTail);
}

template <int CG, bool QRES>
static cudaError_t launch_umma_variant(const UmmaParams& p, cudaStream_t st) {
  const dim3 grid((unsigned)(p.n_part * p.n_query_tiles));
  // pairs and resident queries load row tiles through the 128-row box
  const CUtensorMap& slab_map = (CG == 2 || QRES) ? p.tmap_slab_half : p.tmap_slab;
  return launch_overlapped(umma_score_topk_kernel<CG, QRES>, grid, dim3(UM_THREADS), (size_t)p.smem_bytes, st, CG, p.tmap_q,
                           slab_map, p.n, p.tile_begin, p.tile_end, p.dim, p.nq, p.k, p.n_query_tiles, p.n_part,
                           p.n_stages, p.queue_cap, p.thr_floor, p.partials, p.pace, p.epoch, p.pace_window,
                           p.seed_maxima, p.seed_flags, p.seed_t0, p.seed_look_cycles, p.dev_status);
}

cudaError_t launch_umma(const UmmaParams& p, cudaStream_t st) {
  if (p.n_stages < 2 || p.n_stages > UM_MAX_STAGES || p.queue_cap < 1) return cudaErrorInvalidValue;
  if (p.cta_group != 1 && p.cta_group != 2) return cudaErrorInvalidValue;
  if (p.cta_group == 2 && (p.n_query_tiles % 2) != 0) return cudaErrorInvalidValue;
  if (p.q_resident && (p.cta_group != 1 || p.n_query_tiles != 1 || p.nq > 64)) return cudaErrorInvalidValue;
  if (umma_smem_bytes(p.cta_group, p.q_resident != 0, p.dim, p.k, p.queue_cap, p.n_stages) > (size_t)p.smem_bytes)
    return cudaErrorInvalidValue;
  if (p.partials == nullptr) return cudaErrorInvalidValue;
  if ((p.seed_maxima == nullptr) != (p.seed_flags == nullptr)) return cudaErrorInvalidValue;
  // seeding inside the launch reads the first seed_t0 tiles of every CTA as full tiles
  if (p.seed_maxima != nullptr &&
      (p.seed_t0 < 1 || p.seed_look_cycles < 0 || p.tile_end - p.tile_begin < (int64_t)p.n_part * p.seed_t0 ||
       (p.tile_begin + (int64_t)p.n_part * p.seed_t0) * UM_RT > p.n))
    return cudaErrorInvalidValue;
  if (p.q_resident) return launch_umma_variant<1, true>(p, st);
  return p.cta_group == 2 ? launch_umma_variant<2, false>(p, st) : launch_umma_variant<1, false>(p, st);
}

}  // namespace icc
