// Tensor-core path: scores = Q x X^T on tcgen05 with the partial top-k fused into the epilogue.
//
// Queries are the MMA M operand (128 per CTA), cache rows the N operand (256 per accumulator),
// the embedding dimension is the K loop in 64-element (128-byte, swizzled) chunks.  With this
// orientation tensor-memory lane i of an accumulator holds the scores of query i against 256
// consecutive cache rows, so the epilogue thread that owns lane i owns query i: its admission
// threshold stays in a register and a score costs one compare unless it enters the list.
//
// Warp roles (192 threads, one CTA per SM):
//   warps 0-3  epilogue: tcgen05.ld the accumulator, filter against the per-query threshold,
//              admit the rare survivors into per-query lists in shared memory
//   warp 4     TMA producer: query chunk (16 KiB) + slab chunk (32 KiB) per ring stage
//   warp 5     MMA issuer (one thread) and tensor-memory owner
// Two 256-column accumulators alternate, so the epilogue of one row tile overlaps the MMAs
// of the next.  CTA (p, t) scores query tile t against row tiles p, p + P, p + 2P, ...
// A second instantiation (MAXIMA) shares producer and MMA code but only records, per query and
// tile, the maxima of four groups of 64 rows: the cheap first step of threshold seeding.
#include <math.h>
#include <string.h>

#include "common.cuh"
#include "kernels.h"
#include "pipeline.cuh"

namespace icc {

constexpr int UM_THREADS = 192;
constexpr int UM_QT = 128;            // queries per CTA (MMA M)
constexpr int UM_RT = 256;            // cache rows per accumulator (MMA N)
constexpr int UM_KC = 64;             // elements per K chunk (128 bytes)
constexpr int UM_A_BYTES = UM_QT * UM_KC * 2;   // 16 KiB
constexpr int UM_B_BYTES = UM_RT * UM_KC * 2;   // 32 KiB
constexpr int UM_STAGE_BYTES = UM_A_BYTES + UM_B_BYTES;
// With CTA pairs (CG = 2) the MMA is 256 x 256: each CTA of the pair stages its own 128 queries
// and only half of the 256 cache rows, so a stage is 32 KiB and each slab byte enters the pair
// once for 256 queries.
template <int CG> __host__ __device__ constexpr int um_stage_bytes() { return UM_A_BYTES + UM_B_BYTES / CG; }
constexpr int UM_MAX_STAGES = 8;
constexpr int UM_TMEM_COLS = 512;
constexpr long long PACE_LIMIT_CYCLES = 100000;   // ~50 us: longest a CTA holds back for a slower sibling

struct UmmaSmemTail {
  uint64_t full[UM_MAX_STAGES];
  uint64_t empty[UM_MAX_STAGES];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
};

// MAXIMA = true is the maxima-only variant (no candidate lists): a separate instantiation, so that
// its code costs the list-keeping variant no registers.
template <int CG, bool MAXIMA>
__global__ void __launch_bounds__(UM_THREADS, 1)
umma_score_topk_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_slab,
                       int64_t n, int64_t tile_begin, int64_t tile_end, int dim, int nq, int k, int n_query_tiles,
                       int n_part, int n_stages, int qcap, const uint64_t* __restrict__ thr_floor_in,
                       uint64_t* __restrict__ partials, unsigned long long* pace, unsigned pace_epoch,
                       int pace_window, float* __restrict__ maxima_out, int* dev_status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int STAGE_BYTES = um_stage_bytes<CG>();
  unsigned char* ring = smem;                                                        // n_stages * STAGE_BYTES
  uint64_t* lists = reinterpret_cast<uint64_t*>(ring + (size_t)n_stages * STAGE_BYTES);  // [128][k]
  uint64_t* queues = lists + (size_t)UM_QT * k;                                      // [128][qcap]
  UmmaSmemTail* tail = reinterpret_cast<UmmaSmemTail*>(queues + (size_t)UM_QT * qcap);
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
  // this launch scores row tiles [tile_begin, tile_end); CTA (part, qt) takes every n_part-th
  const int n_kc = (dim + UM_KC - 1) / UM_KC;

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&tail->full[s], CG);       // one arrive.expect_tx per producing CTA
      mbar_init(&tail->empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&tail->acc_full[b], 1);
      mbar_init(&tail->acc_empty[b], 4 * CG);  // one arrival per epilogue warp of every CTA
    }
    mbar_init(&tail->drain, 1);
    tail->abort_flag = 0;
    mbar_fence_init();
  }
  for (int i = tid; i < UM_QT * k; i += UM_THREADS) lists[i] = KEY_EMPTY;
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
      // Pacing.  The CTAs (or pairs) that score different query tiles against the same
      // partition read the same row tiles; the tile comes from HBM once only while they stay
      // within an L2-sized window of each other.  Each publishes how many tiles it has started
      // and one that runs more than pace_window tiles ahead of the slowest holds its loads
      // for a bounded time.  This is a bandwidth hint only: when the bound runs out it goes on.
      const bool paced = (pace != nullptr) && units_per_part > 1 && rank == 0;
      volatile unsigned long long* pace_row = paced ? pace + (size_t)part * units_per_part : nullptr;
      const int my_unit = unit % units_per_part;
      uint32_t ordinal = 0;
      for (int64_t tile = tile_begin + part; tile < tile_end && ok; tile += n_part, ++ordinal) {
        if (paced) pace_row[my_unit] = ((unsigned long long)pace_epoch << 32) | ordinal;
        for (int kc = 0; kc < n_kc; ++kc, ++it) {
          ok = mbar_wait(&tail->empty[s], ph ^ 1u, abort_flag);
          if (!ok) break;
          if (paced && kc == 0) {
            const long long t0 = clock64();
            while (true) {
              uint32_t slowest = ordinal;
              for (int u = 0; u < units_per_part; ++u) {
                const unsigned long long v = pace_row[u];
                const uint32_t o = ((uint32_t)(v >> 32) == pace_epoch) ? (uint32_t)v : 0u;   // not started yet
                slowest = o < slowest ? o : slowest;
              }
              if (ordinal - slowest <= (uint32_t)pace_window || clock64() - t0 > PACE_LIMIT_CYCLES) break;
              __nanosleep(200);
            }
          }
          unsigned char* a_dst = ring + (size_t)s * STAGE_BYTES;
          if (CG == 2) {
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
      if (!ok) {
        report_status(dev_status, DEV_TIMEOUT_MBAR);
        // loads already issued still write this CTA's shared memory: wait for them (bounded)
        for (int64_t j = (it > n_stages ? it - n_stages : 0); j < it && rank == 0; ++j) {
          const int s = (int)(j % n_stages);   // (failure path only)
          const long long t0 = clock64();
          while (!mbar_try_wait(&tail->full[s], (uint32_t)((j / n_stages) & 1)) &&
                 clock64() - t0 < WAIT_LIMIT_CYCLES) {
          }
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(UM_QT * CG, UM_RT);
      int s = 0;          // ring stage and parity as plain counters (see the producer)
      uint32_t ph = 0;
      int64_t lt = 0;
      bool ok = true;
      const uint32_t ring_addr = smem_u32(ring);
      for (int64_t tile = tile_begin + part; tile < tile_end && ok; tile += n_part, ++lt) {
        const int buf = (int)(lt & 1);
        const uint32_t bph = (uint32_t)((lt >> 1) & 1);
        ok = mbar_wait(&tail->acc_empty[buf], bph ^ 1u, abort_flag);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * UM_RT);
        for (int kc = 0; kc < n_kc; ++kc) {
          ok = mbar_wait(&tail->full[s], ph, abort_flag);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t a_addr = ring_addr + (uint32_t)(s * STAGE_BYTES);
          const uint64_t da = umma_desc_k_major_sw128(a_addr);
          const uint64_t db = umma_desc_k_major_sw128(a_addr + UM_A_BYTES);
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
    // Thread t owns query qt*128 + t (tensor-memory lane t).  Its k best candidates live in an
    // unsorted private list in shared memory, stored transposed ([k][32] per warp) so that the
    // 32 lanes of a warp touch 32 consecutive 8-byte words.  The admission threshold (smallest
    // key of the list, its score and its position) stays in registers.
    // A score that passes the threshold is only appended to the thread's small queue (cheap,
    // so lanes that hit in different columns cost little when the warp serialises them); the
    // queues are drained with all lanes working on their own list at the same time: admitting
    // a candidate overwrites the list's smallest entry and rescans the k entries for the new
    // smallest.
    const int q = qt * UM_QT + tid;
    const bool real = q < nq;
    uint64_t* warp_lists = lists + (size_t)(warp * 32) * k;
    uint64_t* my_list = warp_lists + lane;                              // entry i at my_list[i * 32]
    uint64_t* my_queue = queues + (size_t)(warp * 32) * qcap + lane;    // entry i at my_queue[i * 32]
    // A seeding pass over a sample of the rows may have established that k entries with keys
    // >= thr_floor exist: nothing at or below that key can be in the final top-k.
    uint64_t thr_floor = (real && thr_floor_in) ? thr_floor_in[q] : KEY_EMPTY;
    uint64_t thr_key = thr_floor;
    float thr_score = !real ? __int_as_float(0x7fc00000)               // NaN never admits
                            : (thr_floor == KEY_EMPTY ? -INFINITY : key_score(thr_floor));
    int cnt = 0;
    // The list is a min-heap (root = entry 0 = smallest kept key): admitting a candidate replaces
    // the root and sifts it down.  An all-empty list is a valid heap, so no fill phase exists.
    // Place `key` at the root of the 4-ary min-heap my_list[0 .. limit) (children of entry i are
    // 4i+1 .. 4i+4) and sift it down; returns the new root, the smallest entry.  Four children
    // per level keep the chain of dependent shared-memory round trips short: log4(k) levels.
    auto sift_down = [&](uint64_t key, int limit) -> uint64_t {
      int pos = 0;
      uint64_t root = key;
      while (true) {
        const int c0 = 4 * pos + 1;
        if (c0 >= limit) break;
        const uint64_t v0 = my_list[c0 * 32];
        const uint64_t v1 = (c0 + 1 < limit) ? my_list[(c0 + 1) * 32] : ~0ull;
        const uint64_t v2 = (c0 + 2 < limit) ? my_list[(c0 + 2) * 32] : ~0ull;
        const uint64_t v3 = (c0 + 3 < limit) ? my_list[(c0 + 3) * 32] : ~0ull;
        const bool b01 = v1 < v0, b23 = v3 < v2;
        const uint64_t m01 = b01 ? v1 : v0, m23 = b23 ? v3 : v2;
        const int i01 = b01 ? c0 + 1 : c0, i23 = b23 ? c0 + 3 : c0 + 2;
        const bool hi = m23 < m01;
        const uint64_t cv = hi ? m23 : m01;
        if (cv >= key) break;
        my_list[pos * 32] = cv;
        if (pos == 0) root = cv;
        pos = hi ? i23 : i01;
      }
      my_list[pos * 32] = key;
      return root;
    };
    // Up to 16 results: the list lives in registers instead (unsorted; slots >= k hold the largest
    // value so they never count).  Admitting replaces one entry equal to the current minimum and
    // takes the minimum again with a compare tree: pure register arithmetic, no chain of
    // dependent shared-memory round trips.
    constexpr int KREG = 16;
    const bool in_regs = k <= KREG;   // warp-uniform
    uint64_t rl[KREG];
#pragma unroll
    for (int i = 0; i < KREG; ++i) rl[i] = (i < k) ? KEY_EMPTY : ~0ull;
    uint64_t rl_min = KEY_EMPTY;
    auto admit_regs = [&](uint64_t key) -> uint64_t {
      bool placed = false;
#pragma unroll
      for (int i = 0; i < KREG; ++i) {
        const bool here = !placed && rl[i] == rl_min;
        rl[i] = here ? key : rl[i];
        placed = placed || here;
      }
      uint64_t t[KREG];
#pragma unroll
      for (int i = 0; i < KREG; ++i) t[i] = rl[i];
#pragma unroll
      for (int w2 = KREG / 2; w2 >= 1; w2 /= 2) {
#pragma unroll
        for (int i = 0; i < w2; ++i) t[i] = t[i + w2] < t[i] ? t[i + w2] : t[i];
      }
      rl_min = t[0];
      return rl_min;
    };
    auto drain = [&]() {
      for (int i = 0; i < cnt; ++i) {
        const uint64_t raw = my_queue[i * 32];   // (score bits << 32) | slot
        const uint64_t key = make_key(__uint_as_float((uint32_t)(raw >> 32)), (uint32_t)raw);
        if (key > thr_key) {
          const uint64_t root = in_regs ? admit_regs(key) : sift_down(key, k);
          thr_key = root > thr_floor ? root : thr_floor;
          thr_score = (thr_key == KEY_EMPTY) ? -INFINITY : key_score(thr_key);
        }
      }
      cnt = 0;
    };
    int64_t lt = 0;
    bool ok = true;
    for (int64_t tile = tile_begin + part; tile < tile_end; tile += n_part, ++lt) {
      const int buf = (int)(lt & 1);
      const uint32_t bph = (uint32_t)((lt >> 1) & 1);
      ok = mbar_wait(&tail->acc_full[buf], bph, abort_flag);
      ok = __all_sync(FULL_MASK, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t t_addr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * UM_RT);
      const int64_t row0 = tile * UM_RT;
      if constexpr (MAXIMA) {
        // Maxima-only launch (full tiles): no candidate lists, just the best score of each group of
        // 64 cache rows for every query.  The k-th largest of such maxima over all CTAs is a floor
        // for the top-k (k different rows score at least that much); the rows are scored again,
        // with that floor, by the launch that follows.
        float mx[UM_RT / 64];
#pragma unroll
        for (int cp = 0; cp < UM_RT / 64; ++cp) {
          uint32_t v[32], w[32];
          tmem_ld_32x32(t_addr + (uint32_t)(cp * 64), v);
          tmem_ld_32x32(t_addr + (uint32_t)(cp * 64 + 32), w);
          tmem_ld_wait();
          float b = -INFINITY;
#pragma unroll
          for (int c = 0; c < 32; ++c) b = fmaxf(b, fmaxf(__uint_as_float(v[c]), __uint_as_float(w[c])));
          mx[cp] = b;
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(lead_acc_empty0 + (uint32_t)(buf * 8));
        if (real)
          *reinterpret_cast<float4*>(maxima_out + ((size_t)(tile - tile_begin) * nq + q) * 4) =
              make_float4(mx[0], mx[1], mx[2], mx[3]);
        continue;
      }
      if (lt == 0 && thr_floor_in == nullptr && k <= 16 && row0 + UM_RT <= n) {
        // Cold start (empty lists, no seed threshold): read the tile once just to take the
        // maximum of each group of 8 columns.  The k-th largest of the 32 group maxima is a
        // safe floor - k different columns score at least that much - and only a few percent
        // of the columns pass it (about 12 of 256 for k = 10, 21 for k = 16), instead of every
        // column passing an empty list.
        float m[32];
#pragma unroll
        for (int cb = 0; cb < UM_RT / 32; ++cb) {
          uint32_t v[32];
          tmem_ld_32x32(t_addr + (uint32_t)(cb * 32), v);
          tmem_ld_wait();
#pragma unroll
          for (int gq = 0; gq < 4; ++gq) {
            float a = __uint_as_float(v[8 * gq]);
#pragma unroll
            for (int c = 1; c < 8; ++c) a = fmaxf(a, __uint_as_float(v[8 * gq + c]));
            m[4 * cb + gq] = a;
          }
        }
        // bitonic sorting network, descending, on registers
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
                  const float hi = fmaxf(m[i], m[j]), lo = fminf(m[i], m[j]);
                  m[i] = desc ? hi : lo;
                  m[j] = desc ? lo : hi;
                }
              }
            }
          }
        }
        // m is sorted descending: its k-th entry is the largest of the entries k-1 .. 31
        float tau = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; ++i) tau = fmaxf(tau, i >= k - 1 ? m[i] : -INFINITY);
        if (real && tau == tau) {
          // admit every key whose score is >= tau: the smallest such key has slot word 0
          thr_floor = ((uint64_t)score_to_ord(tau) << 32) - 1;
          thr_key = thr_floor;
          thr_score = tau;
        }
      }
      // Tensor-memory loads take several hundred cycles each while MMAs are running, so the tile
      // is read 64 columns at a time with two loads in flight, and one vote rejects all 64 columns
      // in the common case.  Only when some lane has a passing column are the two halves taken
      // through the admission code below, one after the other.
#pragma unroll 1
      for (int cp = 0; cp < UM_RT / 64; ++cp) {
        uint32_t v[32], w[32];
        tmem_ld_32x32(t_addr + (uint32_t)(cp * 64), v);
        tmem_ld_32x32(t_addr + (uint32_t)(cp * 64 + 32), w);
        tmem_ld_wait();
        if (cp == UM_RT / 64 - 1) {
          // the accumulator has been read completely: hand it back to the MMA issuer
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(lead_acc_empty0 + (uint32_t)(buf * 8));
        }
        if (row0 + cp * 64 + 64 <= n) {   // warp-uniform; a ragged tail goes through the per-half masks
          float b[8];
#pragma unroll
          for (int j = 0; j < 8; ++j)
            b[j] = fmaxf(fmaxf(fmaxf(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1])),
                               fmaxf(__uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]))),
                         fmaxf(fmaxf(__uint_as_float(w[4 * j]), __uint_as_float(w[4 * j + 1])),
                               fmaxf(__uint_as_float(w[4 * j + 2]), __uint_as_float(w[4 * j + 3]))));
          const float best64 = fmaxf(fmaxf(fmaxf(b[0], b[1]), fmaxf(b[2], b[3])), fmaxf(fmaxf(b[4], b[5]), fmaxf(b[6], b[7])));
          if (!__any_sync(FULL_MASK, best64 >= thr_score)) continue;
        }
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
          if (h == 1) {
#pragma unroll
            for (int c = 0; c < 32; ++c) v[c] = w[c];
          }
          const int cb = cp * 2 + h;
          const int64_t col0 = row0 + cb * 32;
          float g[8];                                   // maxima of the eight groups of four columns
          bool active = col0 < n;                       // warp-uniform
          if (active) {
            if (n - col0 < 32) {                        // ragged last tile: columns past n never admit
#pragma unroll
              for (int c = 0; c < 32; ++c)
                if (col0 + c >= n) v[c] = 0x7fc00000u;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
              g[j] = fmaxf(fmaxf(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1])),
                           fmaxf(__uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
            const float best = fmaxf(fmaxf(fmaxf(g[0], g[1]), fmaxf(g[2], g[3])), fmaxf(fmaxf(g[4], g[5]), fmaxf(g[6], g[7])));
            active = __any_sync(FULL_MASK, best >= thr_score);   // common case: nothing passes
          }
          // Common slow case: every lane's queue has room for all of its passing columns.  One
          // vote establishes that, one OR-reduction tells which groups of columns anybody needs,
          // and the pushes are predicated stores: no per-group votes, no divergent branches.
          bool drain_after = false;
          if (active) {
            uint32_t hm = 0;
#pragma unroll
            for (int c = 0; c < 32; ++c) hm |= (__uint_as_float(v[c]) >= thr_score) ? (1u << c) : 0u;
            if (!__any_sync(FULL_MASK, cnt + __popc(hm) > qcap)) {
              const uint32_t cols = __reduce_or_sync(FULL_MASK, hm);
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                if ((cols >> (4 * j)) & 0xfu) {   // warp-uniform
#pragma unroll
                  for (int c = 4 * j; c < 4 * j + 4; ++c) {
                    if ((hm >> c) & 1u) {
                      my_queue[cnt * 32] = ((uint64_t)v[c] << 32) | (uint32_t)(col0 + c);
                      ++cnt;
                    }
                  }
                }
              }
              active = false;
              drain_after = __any_sync(FULL_MASK, 2 * cnt >= qcap);
            }
          }
          // Otherwise (cold start, very loose thresholds): warp-uniform control flow with the queue
          // drained at one place only (the code stays small and a drain is always entered by all
          // 32 lanes, each working through its own queue).  Columns are considered in order;
          // whenever some lane's queue could not take another group of four (or, for queues
          // shorter than four, another entry) the pass stops, the queues are drained and the pass
          // resumes at c_next.
          int c_next = 0;
          while (true) {
            bool need_drain = drain_after;
            drain_after = false;
            if (active) {
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                if (!need_drain && 4 * j + 3 >= c_next && __any_sync(FULL_MASK, g[j] >= thr_score)) {
#pragma unroll
                  for (int c = 4 * j; c < 4 * j + 4; ++c) {
                    if (!need_drain && c >= c_next) {
                      const float s = __uint_as_float(v[c]);
                      if (s >= thr_score) {
                        my_queue[cnt * 32] = ((uint64_t)v[c] << 32) | (uint32_t)(col0 + c);
                        ++cnt;
                      }
                      if (qcap < 4 && __any_sync(FULL_MASK, cnt >= qcap)) {
                        need_drain = true;
                        c_next = c + 1;
                      }
                    }
                  }
                  if (!need_drain && qcap >= 4 && __any_sync(FULL_MASK, cnt + 4 > qcap)) {
                    need_drain = true;
                    c_next = 4 * j + 4;
                  }
                }
              }
              if (!need_drain) {
                active = false;
                need_drain = __any_sync(FULL_MASK, 2 * cnt >= qcap);
              }
            }
            if (need_drain) drain();
            if (!active) break;
          }
        }   // halves
      }
      // fresh thresholds for the next tile
      if (__any_sync(FULL_MASK, cnt > 0)) drain();
    }
    if (!ok && lane == 0) report_status(dev_status, DEV_TIMEOUT_MBAR);
    if constexpr (MAXIMA) {
      // nothing to sort or write: this launch produced maxima only
    } else if (in_regs) {
      // sort the register list descending with a bitonic network (the padding slots >= k hold the
      // largest value: turn them into the smallest first so that they sort to the end)
#pragma unroll
      for (int i = 0; i < KREG; ++i) rl[i] = (i < k) ? rl[i] : KEY_EMPTY;
#pragma unroll
      for (int ls = 1; ls <= 4; ++ls) {
#pragma unroll
        for (int lj = 3; lj >= 0; --lj) {
          if (lj < ls) {
#pragma unroll
            for (int i = 0; i < KREG; ++i) {
              const int j = i ^ (1 << lj);
              if (j > i) {
                const bool desc = (i & (1 << ls)) == 0;
                const uint64_t hi = rl[i] > rl[j] ? rl[i] : rl[j], lo = rl[i] > rl[j] ? rl[j] : rl[i];
                rl[i] = desc ? hi : lo;
                rl[j] = desc ? lo : hi;
              }
            }
          }
        }
      }
#pragma unroll
      for (int i = 0; i < KREG; ++i)
        if (i < k) my_list[i * 32] = rl[i];
    } else {
      // sort each private list descending, lanes in parallel: heapsort in place (the smallest
      // entry goes to the end of the shrinking heap)
      for (int end = k - 1; end > 0; --end) {
        const uint64_t smallest = my_list[0];
        const uint64_t moved = my_list[end * 32];
        my_list[end * 32] = smallest;
        sift_down(moved, end);
      }
    }
    __syncwarp();
    // transpose out: the partial lists of this warp's queries are contiguous in global memory
    const int q_first = qt * UM_QT + warp * 32;
    const int q_live = min(32, nq - q_first);
    if (q_live > 0 && !MAXIMA) {
      uint64_t* dst = partials + ((size_t)part * nq + q_first) * k;
      for (int i = lane; i < q_live * k; i += 32) {
        const int ql = i / k, e = i - ql * k;
        dst[i] = warp_lists[e * 32 + ql];
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
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(umma_score_topk_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  return e;
}

template <int CG, bool MAXIMA>
static cudaError_t launch_umma_variant(const UmmaParams& p, cudaStream_t st) {
  const dim3 grid((unsigned)(p.n_part * p.n_query_tiles));
  return launch_overlapped(umma_score_topk_kernel<CG, MAXIMA>, grid, dim3(UM_THREADS), (size_t)p.smem_bytes, st, CG, p.tmap_q,
                           CG == 2 ? p.tmap_slab_half : p.tmap_slab, p.n, p.tile_begin, p.tile_end, p.dim, p.nq, p.k,
                           p.n_query_tiles, p.n_part, p.n_stages, p.queue_cap, p.thr_floor, p.partials, p.pace,
                           p.pace_epoch, p.pace_window, p.maxima_out, p.dev_status);
}

cudaError_t launch_umma(const UmmaParams& p, cudaStream_t st) {
  if (p.n_stages < 2 || p.n_stages > UM_MAX_STAGES || p.queue_cap < 1) return cudaErrorInvalidValue;
  if (p.cta_group != 1 && p.cta_group != 2) return cudaErrorInvalidValue;
  if (p.cta_group == 2 && (p.n_query_tiles % 2) != 0) return cudaErrorInvalidValue;
  const int stage_bytes = p.cta_group == 2 ? um_stage_bytes<2>() : um_stage_bytes<1>();
  const size_t need = 1024 + (size_t)p.n_stages * stage_bytes + (size_t)UM_QT * (p.k + p.queue_cap) * 8 + sizeof(UmmaSmemTail);
  if (need > (size_t)p.smem_bytes) return cudaErrorInvalidValue;
  if (p.maxima_out != nullptr) {
    // maxima-only launches cover full tiles only
    if (p.tile_end * UM_RT > p.n) return cudaErrorInvalidValue;
    return p.cta_group == 2 ? launch_umma_variant<2, true>(p, st) : launch_umma_variant<1, true>(p, st);
  }
  if (p.partials == nullptr) return cudaErrorInvalidValue;
  return p.cta_group == 2 ? launch_umma_variant<2, false>(p, st) : launch_umma_variant<1, false>(p, st);
}

}  // namespace icc
