// Tensor-core scoring for 16-bit inputs on sm_100a: one persistent kernel that
// computes the accumulated SG-softmax score (Eq. 1, 5, 9) of every KV head and,
// on the way, the squared value norms of Section 4.3.
//
// Work unit: a "row block" = up to 128 stacked observation rows (query heads of
// one KV head x observation rows) against all n keys, cut into 128-key tiles.
// A normalised column sum needs each row's softmax statistics over ALL keys
// first, so every tile is visited twice:
//
//   pass 1 (rows on TMEM lanes):  D = Q . K^T   -> per-row log2 sum of 2^{c w} over a run of
//                                 tiles, stored to global memory as one 4-byte partial
//                                 per row and run.
//   pass 2 (keys on TMEM lanes):  D = K . Q^T - off/c -> each thread owns one key and adds
//                                 2^{c D} over the rows: the column sum needs no
//                                 cross-thread traffic and no per-row constant but c.
//
// Both products are tcgen05.mma kind::f16 with FP32 accumulators in TMEM, fed by
// TMA (128-byte swizzle) from the same K-major Q and K tiles, which serve as A or
// B operand alike.
//
// Schedule.  A run is up to CH consecutive key tiles of one row block.  Runs are handed out to the CTAs
// as they come free, from two global counters: one for pass 1, one for pass 2.  The TMA thread of
// every CTA takes one run of each per round (pass 2 only once every pass-1 run of that row block has been
// taken by somebody) and publishes the CTA's sequence of segments, P1(a), P2(b), P1(a'), P2(b'), ..., in a
// ring in shared memory that all other roles read in order; the pass-2 run of a round is announced to the
// merge group a round early.  One pipeline serves the sequence: one TMA warp, one MMA warp, a ring of K
// tiles, four TMEM accumulators and sixteen softmax warps that take whichever kind of tile comes next.
// Pass 2 trails pass 1 by about one round of the whole grid: long enough for every CTA to have delivered
// its share of a row block's statistics, short enough for the keys to be still in L2, so that HBM sees K
// once.  SMs that fall behind simply take fewer runs.
//
// Between the passes there are no flags, counters or fences.  The partials start
// as NaN (the host clears them before the launch) and each is published by a single
// 4-byte store, so a reader knows a partial is there when it no longer reads NaN.
// Every CTA merges, for the run its pass 2 turns to next, the partials of all
// runs of that row block into one offset per row by itself (two warps do this up to
// two runs ahead of the MMAs, off the critical path), always in run order: the
// result does not depend on who finished first.
//
// The row offsets ride in the product itself: the merged offset of a row becomes
// -off/(2 c kFold) as a sum of three 16-bit numbers, written twice into a 16-element
// extension of the row in shared memory, and pass 2 appends one more k-step of the
// MMA that multiplies the extension with a constant tile holding kFold.  The three
// parts carry 24 (bfloat16) or 33 (float16) significant bits, the products are exact
// and the accumulator is FP32, so D = w - off/c to FP32 rounding.  Both 16-byte
// halves of a row are identical in either tile, so the result does not depend on how
// the 32-byte swizzle orders them.
//
// The value rows of the keys of each pass-1 tile stream through a small ring of their
// own (evict-first in L2); four warps square and add them: nu_j = |V_j|^2 costs no
// launch and no second sweep of HBM.
//
// The kernel is launched cooperatively with at most one CTA per SM, which guarantees
// that the CTAs a partial comes from are running; a segment only ever waits for
// segments that were handed out before it, so the waits cannot deadlock.  Every wait is
// bounded in time; on expiry the kernel records AHAKV_ERR_TIMEOUT in the status word
// and winds down.
#include <cuda.h>

#include <atomic>

#include "ahakv_internal.cuh"
#include "tc_common.cuh"

namespace ahakv {
namespace {

using namespace tc;

constexpr int kKStages = 3;                // K-tile ring depth
constexpr int kSubTileBytes = 128 * 128;   // 128 rows x 64 16-bit elements, 128-byte swizzled
constexpr int kVRows = 64;                 // value rows per V-ring stage
constexpr int kVStages = 2;
constexpr int kSegRing = 64;               // published segments a role may lag behind the scheduler
constexpr int kMergeRing = 8;
constexpr int kSegAhead = 4;               // segments published beyond the one the softmax warps are on
constexpr int kSegEnd = -1;
constexpr int kVSubBytes = kVRows * 128;
constexpr int kThreads = 768;              // TMA + scheduler warp, MMA warp, 2 merge warps, 16 softmax warps, 4 value-norm warps
constexpr float kFold = 256.f;             // value of the constant tile; offsets are stored divided by it

struct TcArgs {
  int n, r, G, Hkv, n_rb, hb, n_blk, D;
  int CH;         // key tiles per run
  int rpu;        // runs per row block = ceil(n_blk / CH)
  int n_runs;     // row blocks * rpu
  int bf16;       // operand type of the products
  int prior;      // stream V and write nu
  float log2G;
  float c[kMaxRows];     // lambda_i log2(e) per observation row
  float cs[128];         // the same per stacked row of a row block (r <= 128 only)
  int last[kMaxRows];    // per observation row: the last key it may see
  int min_last;          // the smallest of them: tiles that end at or before it are masked for no row
  float* partial;    // [unit][run][128]: log2 of a row's sum of 2^{c w} over the run's keys
  float* s_raw;      // [unit][n]
  float* nu;         // [B * Hkv][n]
  int* ctr;          // [2] next pass-1 run, next pass-2 run (zero at launch)
  int* status;
  long long test_wait_ns;   // test build of the kernel only: what every bounded wait allows
  int test_withhold;        // test build only: the partial of the first run of the first row block is never published
};

// The kernel exists twice: the one every call runs, whose waits allow kWaitLimitNs, and a second instantiation that
// takes the limit and a planted fault from its arguments, for the test of the failure path (ahakv_test_set_wait).
// Same code, same wind-down; only these two lines differ.
template <bool kTest> __device__ __forceinline__ long long wait_limit(const TcArgs& a) {
  return kTest ? a.test_wait_ns : kWaitLimitNs;
}

// ---- shared memory layout --------------------------------------------------------------------
struct __align__(8) Barriers {
  unsigned long long q_full[2], q_empty[2];
  unsigned long long k_full[kKStages], k_empty[kKStages];
  unsigned long long v_full[kVStages], v_empty[kVStages];
  unsigned long long acc_full[4], acc_empty[4];
  unsigned long long ext_full[2], ext_empty[2];   // offset extension of a run's row block: merge group -> MMA
};

struct Shared {
  Barriers bars;
  uint32_t tmem_slot;
  int seg_pub, seg_done_soft, seg_done_v;   // segments published / retired by the softmax warps / by the value-norm warps
  int mrg_pub, mrg_done;                    // pass-2 runs announced to / finished by the merge group
  int seg[kSegRing];                        // 2 * run + pass, or kSegEnd
  int mrg[kMergeRing];                      // run, or kSegEnd
  float c[kMaxRows];            // lambda_i * log2(e) per observation row
  float cs2[2][128];            // c per stacked row, by row block parity (r > 128 has two kinds of block)
  int vis_off[2][128];          // per stacked row: the last key its observation row may see
  float2 p1_part[2][3][128];    // pass 1: statistics of the three groups that do not publish
  float p2_part[2][3][128];     // pass 2: partial column sums of the three groups that do not store
};

constexpr int kQBytes = 2 * kSubTileBytes;              // D <= 128
constexpr int kKStageBytes = 2 * kSubTileBytes;
constexpr int kVStageBytes = 2 * kVSubBytes;
constexpr int kExtBytes = 128 * 32;                      // 128 rows x 16 16-bit elements, 32-byte swizzled
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + 2 * kQBytes;
constexpr int kOffV = kOffK + kKStages * kKStageBytes;
constexpr int kOffExt = kOffV + kVStages * kVStageBytes;        // two extensions, then the constant tile
constexpr int kSmemTiles = kOffExt + 3 * kExtBytes;      // 204 KiB
constexpr int kSmemBytes = kSmemTiles + 1024 /*alignment slack*/ + 13312 /*barriers, constants, exchange*/;
static_assert(sizeof(Shared) <= 13312, "Shared outgrew its reservation");

// ---- work decomposition ----------------------------------------------------------------------------------
// A run = up to CH consecutive key tiles of one row block.  Every role of a CTA walks the runs its scheduler
// has taken, in the order of the CTA's segment ring.
struct Run {
  int unit, rin, blk0, cnt;
};
__device__ __forceinline__ Run run_info(const TcArgs& a, int run) {
  Run r;
  r.unit = run / a.rpu;
  r.rin = run % a.rpu;
  r.blk0 = r.rin * a.CH;
  r.cnt = min(a.CH, a.n_blk - r.blk0);
  return r;
}

struct UnitInfo {
  int unit, bh, rb, b, h, rows, npad;
};
__device__ __forceinline__ UnitInfo unit_info(const TcArgs& a, int unit) {
  UnitInfo u;
  u.unit = unit;
  u.bh = unit / a.n_rb;
  u.rb = unit % a.n_rb;
  u.b = u.bh / a.Hkv;
  u.h = u.bh % a.Hkv;
  // r <= 128: hb query heads a block, fewer in the last block of a KV head when hb does not divide G (the
  // box still brings hb heads' rows; those past `rows` belong to another KV head or read as zeros, and no
  // result depends on them)
  u.rows = a.r <= 128 ? min(a.hb, a.G - u.rb * a.hb) * a.r : min(128, a.r - u.rb * 128);
  u.npad = (u.rows + 15) & ~15;
  return u;
}
// Observation row index (0 .. r-1) of stacked row s of a row block.
__device__ __forceinline__ int obs_row(const TcArgs& a, const UnitInfo& u, int s) {
  return a.r <= 128 ? s % a.r : u.rb * 128 + s;
}

// ---- the CTA's sequence of segments -------------------------------------------------------------------
__device__ __forceinline__ int ld_volatile(const int* p) { return *(const volatile int*)p; }

// Entry `idx` of the sequence if the scheduler has published it, else -2.
__device__ __forceinline__ int seg_peek(Shared* sh, int idx) {
  if (idx >= ld_volatile(&sh->seg_pub)) return -2;
  __threadfence_block();
  return ld_volatile(&sh->seg[idx % kSegRing]);
}
// The same, waiting (bounded) for the scheduler.  kSegEnd ends the sequence; so does a wait that ran out.
// Readers allow twice the time the scheduler's own thread does: when nothing moves, that thread gives up first and
// publishes kSegEnd, so every reader of the CTA sees the same end of the sequence rather than its own.
__device__ __forceinline__ int seg_get(Shared* sh, int idx, int* status, long long limit_ns) {
  int e = seg_peek(sh, idx);
  if (e != -2) return e;
  long long t0 = -1;
  for (int spins = 0;; ++spins) {
    __nanosleep(64);
    if ((e = seg_peek(sh, idx)) != -2) return e;
    if ((spins & 255) != 255) continue;                   // the clock is slow to read
    if (t0 < 0) t0 = now_ns();
    else if (now_ns() - t0 > 2 * limit_ns) {
      atomicExch(status, (int)AHAKV_ERR_TIMEOUT);
      return kSegEnd;
    }
  }
}
__device__ __forceinline__ int mrg_get(Shared* sh, int idx, int* status, long long limit_ns) {
  const long long t0 = now_ns();
  for (;;) {
    if (idx < ld_volatile(&sh->mrg_pub)) {
      __threadfence_block();
      return ld_volatile(&sh->mrg[idx % kMergeRing]);
    }
    __nanosleep(200);
    if (now_ns() - t0 > 2 * limit_ns) {
      atomicExch(status, (int)AHAKV_ERR_TIMEOUT);
      return kSegEnd;
    }
  }
}

// f(pass, run) for every segment of this CTA, in order.
template <bool kTest, typename F>
__device__ __forceinline__ void for_each_segment(const TcArgs& a, Shared* sh, F f) {
  for (int idx = 0;; ++idx) {
    const int e = seg_get(sh, idx, a.status, wait_limit<kTest>(a));
    if (e == kSegEnd) return;
    f(e & 1, e >> 1, idx);
  }
}

// Scheduler state of a CTA (kept by its TMA thread): hands the CTA its runs.  A round takes the next pass-1
// run and publishes it; publishes the pass-2 run taken in an earlier round -- only once every pass-1 run of
// its row block has been taken by somebody, so that whoever waits for that block's statistics waits for work
// that is already under way; then takes the next pass-2 run and announces it to the merge group.
struct Scheduler {
  int k, m, pend;
  bool p1_left, p2_left, done;
};
__device__ __forceinline__ void sched_publish(Shared* sh, Scheduler& sc, int entry) {
  sh->seg[sc.k % kSegRing] = entry;
  __threadfence_block();
  *(volatile int*)&sh->seg_pub = ++sc.k;
}
__device__ __forceinline__ void sched_announce(Shared* sh, Scheduler& sc, int run) {
  sh->mrg[sc.m % kMergeRing] = run;
  __threadfence_block();
  *(volatile int*)&sh->mrg_pub = ++sc.m;
}
// One round, if there is room for it (never waits).  Returns whether anything was published.
__device__ bool sched_round(const TcArgs& a, Shared* sh, Scheduler& sc) {
  if (sc.done) return false;
  const int ds = ld_volatile(&sh->seg_done_soft), dv = ld_volatile(&sh->seg_done_v);
  // room in both rings for a whole round, and not too far ahead of the tiles being worked on
  if (sc.k - (ds < dv ? ds : dv) > kSegRing - 4 || sc.k - ds >= kSegAhead ||
      sc.m - ld_volatile(&sh->mrg_done) > kMergeRing - 2)
    return false;
  bool did = false;
  if (sc.p1_left) {
    const int r = atomicAdd(&a.ctr[0], 1);
    if (r < a.n_runs) { sched_publish(sh, sc, 2 * r); did = true; }
    else sc.p1_left = false;
  }
  if (sc.pend >= 0) {
    // the pass-2 run in hand joins the sequence once all pass-1 runs of its row block have been taken
    const int need = min((sc.pend / a.rpu + 1) * a.rpu, a.n_runs);
    if (ld_volatile(&a.ctr[0]) >= need) { sched_publish(sh, sc, 2 * sc.pend + 1); sc.pend = -1; did = true; }
  }
  if (sc.pend < 0 && sc.p2_left) {
    const int b = atomicAdd(&a.ctr[1], 1);
    if (b < a.n_runs) { sc.pend = b; sched_announce(sh, sc, b); did = true; }
    else sc.p2_left = false;
  }
  if (!sc.p1_left && !sc.p2_left && sc.pend < 0) {
    sched_announce(sh, sc, kSegEnd);
    sched_publish(sh, sc, kSegEnd);
    sc.done = true;
    did = true;
  }
  return did;
}

// The next 64 value rows to fetch or to square: stage t of a pass-1 segment (first row block of a KV head
// only).  `idx` walks the CTA's sequence.
struct VCursor {
  int idx, t, cnt, row0, b, h, bh;
};
// Moves to the first stage of the next segment that brings value rows.  1: found, 0: the sequence has ended,
// -1: not published yet (only when `block` is false).
template <bool kTest>
__device__ __forceinline__ int v_seek(const TcArgs& a, Shared* sh, VCursor& c, bool block, int* behind = nullptr) {
  for (;; ++c.idx) {
    if (behind) *(volatile int*)behind = c.idx;               // everything before c.idx has been dealt with
    const int e = block ? seg_get(sh, c.idx, a.status, wait_limit<kTest>(a)) : seg_peek(sh, c.idx);
    if (e == -2) return -1;
    if (e == kSegEnd) return 0;
    if (e & 1) continue;
    const Run rn = run_info(a, e >> 1);
    const UnitInfo u = unit_info(a, rn.unit);
    if (u.rb != 0) continue;
    c.t = 0; c.cnt = 2 * rn.cnt; c.row0 = rn.blk0 * kKeyTile; c.b = u.b; c.h = u.h; c.bh = u.bh;
    return 1;
  }
}

// ---- roles --------------------------------------------------------------------------------------------
// TMA producer: one thread keeps the CTA's sequence of segments filled (scheduler rounds) and feeds two
// independent streams, whichever has a free slot: Q and K tiles in the order of the sequence, and the value
// rows that go with the pass-1 key tiles.
template <bool kTest>
__device__ void producer(const TcArgs& a, const CUtensorMap* qmap, const CUtensorMap* kmap, const CUtensorMap* vmap,
                         Shared* sh, char* tiles) {
  Barriers* bars = &sh->bars;
  const int n_sub = a.D / 64;
  const int q_rows = a.r <= 128 ? a.hb * a.r : 128;
  const int q_bytes = n_sub * q_rows * 128, k_bytes = n_sub * kSubTileBytes;
  const unsigned long long once = policy_evict_first();

  // K stream state: 0 waiting for the next segment, 1 Q to load, 2 tiles to load, 3 done
  int k_state = 0, k_idx = 0, pass = 0, tc = 0, sc = 0, t = 0;
  Run rn = run_info(a, 0);
  UnitInfo u = unit_info(a, 0);
  // V stream state: 0 waiting for the next segment with value rows, 2 stages to load, 3 done
  VCursor vcur;
  vcur.idx = 0;
  int v_state = a.prior ? 0 : 3, vc = 0;

  Scheduler sched = {0, 0, -1, true, true, false};
  long long idle_since = -1;
  int idle_spins = 0;
  while (k_state != 3 || v_state != 3) {
    bool progress = false;
    // a new round whenever the K stream is about to run dry
    if (k_state == 0 && seg_peek(sh, k_idx) == -2) progress = sched_round(a, sh, sched);
    if (k_state == 0) {
      const int e = seg_peek(sh, k_idx);
      if (e == kSegEnd) { k_state = 3; progress = true; }
      else if (e != -2) {
        ++k_idx;
        pass = e & 1;
        rn = run_info(a, e >> 1);
        u = unit_info(a, rn.unit);
        t = 0;
        k_state = 1;
        progress = true;
      }
    }
    if (k_state == 1) {
      const int qb = sc & 1;
      if (mbar_try(&bars->q_empty[qb], ((sc >> 1) & 1) ^ 1)) {
        char* q_smem = tiles + kOffQ + qb * kQBytes;
        mbar_expect_tx(&bars->q_full[qb], q_bytes);
        for (int s = 0; s < n_sub; ++s) {
          if (a.r <= 128) tma_load_4d(q_smem + s * kSubTileBytes, qmap, &bars->q_full[qb], s * 64, 0, u.h * a.G + u.rb * a.hb, u.b);
          else tma_load_4d(q_smem + s * kSubTileBytes, qmap, &bars->q_full[qb], s * 64, u.rb * 128, u.h, u.b);
        }
        ++sc;
        k_state = 2;
        progress = true;
      }
    } else if (k_state == 2) {
      const int stage = tc % kKStages, ph = (tc / kKStages) & 1;
      if (mbar_try(&bars->k_empty[stage], ph ^ 1)) {
        mbar_expect_tx(&bars->k_full[stage], k_bytes);
        char* dst = tiles + kOffK + stage * kKStageBytes;
        for (int s = 0; s < n_sub; ++s) {
          // the second read of a key tile is its last: let L2 drop it first
          if (pass == 0) tma_load_4d(dst + s * kSubTileBytes, kmap, &bars->k_full[stage], s * 64, (rn.blk0 + t) * kKeyTile, u.h, u.b);
          else tma_load_4d_hint(dst + s * kSubTileBytes, kmap, &bars->k_full[stage], s * 64, (rn.blk0 + t) * kKeyTile, u.h, u.b, once);
        }
        ++tc;
        if (++t == rn.cnt) k_state = 0;
        progress = true;
      }
    }
    if (v_state == 0) {
      const int f = v_seek<kTest>(a, sh, vcur, false);
      if (f == 1) { v_state = 2; progress = true; }
      else if (f == 0) { v_state = 3; progress = true; }
    }
    if (v_state == 2) {
      const int vs = vc % kVStages;
      if (mbar_try(&bars->v_empty[vs], ((vc / kVStages) & 1) ^ 1)) {
        mbar_expect_tx(&bars->v_full[vs], n_sub * kVSubBytes);
        char* dst = tiles + kOffV + vs * kVStageBytes;
        for (int s = 0; s < n_sub; ++s)
          tma_load_4d_hint(dst + s * kVSubBytes, vmap, &bars->v_full[vs], s * 64, vcur.row0 + vcur.t * kVRows, vcur.h, vcur.b, once);
        ++vc;
        if (++vcur.t == vcur.cnt) { ++vcur.idx; v_state = 0; }
        progress = true;
      }
    }
    if (progress) {
      idle_since = -1;
      idle_spins = 0;
    } else if ((++idle_spins & 1023) == 0) {               // the clock is slow to read: look at it rarely
      const long long now = now_ns();
      if (idle_since < 0) idle_since = now;
      else if (now - idle_since > wait_limit<kTest>(a)) {
        atomicExch(a.status, (int)AHAKV_ERR_TIMEOUT);
        if (!sched.done) { sched_announce(sh, sched, kSegEnd); sched_publish(sh, sched, kSegEnd); }
        // wind down: give copies already in flight a bounded time (1 ms) to land before the CTA exits
        while (now_ns() - now < 1000000) __nanosleep(1000);
        return;
      }
    }
  }
}

// Value-norm group (four warps, 128 threads): two adjacent lanes share a row of each 64-row stage of the
// V ring (one half of its 16-byte chunks each, in an order that keeps them on different banks), square
// and add in FP32 and meet by shuffle: nu_j = |V_j|^2.
template <bool kTest>
__device__ void v_group(const TcArgs& a, Shared* sh, char* tiles) {
  Barriers* bars = &sh->bars;
  const int row = (threadIdx.x & 127) >> 1, sub = threadIdx.x & 1;
  const bool leader = (threadIdx.x & 127) == 0;
  VCursor cc;
  cc.idx = 0;
  int ci = 0;
  while (v_seek<kTest>(a, sh, cc, true, leader ? &sh->seg_done_v : nullptr) == 1) {
    for (; cc.t < cc.cnt; ++cc.t, ++ci) {
      const int vs = ci % kVStages;
      if (!mbar_wait(&bars->v_full[vs], (ci / kVStages) & 1, a.status, wait_limit<kTest>(a))) return;
      const char* stage = tiles + kOffV + vs * kVStageBytes;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        // head_dim 128: lane `sub` takes sub-tile `sub`, chunks in the order c ^ sub; head_dim 64: chunks
        // 4 sub .. 4 sub + 3 of the one sub-tile
        const int chunk = a.D == 128 ? (c ^ sub) : (4 * sub + c);
        if (a.D == 128 || c < 4) {
          const uint4 q = *reinterpret_cast<const uint4*>(stage + (a.D == 128 ? sub * kVSubBytes : 0) + row * 128 +
                                                          ((chunk ^ (row & 7)) << 4));
          float f[8];
          if (a.bf16) Vec16<__nv_bfloat16>::widen(q, f);
          else Vec16<__half>::widen(q, f);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e & 3] = fmaf(f[e], f[e], acc[e & 3]);
        }
      }
      mbar_arrive(&bars->v_empty[vs]);
      float sq = (acc[0] + acc[1]) + (acc[2] + acc[3]);
      sq += __shfl_xor_sync(0xffffffffu, sq, 1);
      const int j = cc.row0 + cc.t * kVRows + row;
      if (sub == 0 && j < a.n) a.nu[(size_t)cc.bh * a.n + j] = sq;
    }
    ++cc.idx;
  }
  if (leader) *(volatile int*)&sh->seg_done_v = 0x3fffffff;
}

// MMA issuer (one thread).
// Pass 1: D[rows x keys] = Q K^T.  Pass 2: D[keys x rows] = K Q^T - off / c.
template <bool kTest>
__device__ void mma_issuer(const TcArgs& a, Shared* sh, char* tiles, uint32_t tmem_base) {
  Barriers* bars = &sh->bars;
  int tc = 0, sc = 0, pc = 0;
  bool ok = true;
  const uint64_t fold_desc = umma_desc_ext(smem_u32(tiles + kOffExt + 2 * kExtBytes));
  const int nk = a.D / 16;
  for_each_segment<kTest>(a, sh, [&](int pass, int run, int) {
    if (!ok) return;
    const Run rn = run_info(a, run);
    const int qb = sc & 1;
    if (!(ok = mbar_wait(&bars->q_full[qb], (sc >> 1) & 1, a.status, wait_limit<kTest>(a)))) return;
    uint32_t idesc = umma_idesc(128, 128, a.bf16);
    uint64_t ext_desc = 0;
    const int slot = pc & 1;
    if (pass == 1) {
      // the row block's offset extension, from this CTA's merge group
      if (!(ok = mbar_wait(&bars->ext_full[slot], (pc >> 1) & 1, a.status, wait_limit<kTest>(a)))) return;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      idesc = umma_idesc(128, unit_info(a, rn.unit).npad, a.bf16);
      ext_desc = umma_desc_ext(smem_u32(tiles + kOffExt + slot * kExtBytes));
    }
    for (int t = 0; t < rn.cnt; ++t, ++tc) {
      const int stage = tc % kKStages, ph = (tc / kKStages) & 1;
      const int acc = tc & 3, aph = (tc >> 2) & 1;      // the four accumulators in turn
      if (!(ok = mbar_wait(&bars->acc_empty[acc], aph ^ 1, a.status, wait_limit<kTest>(a)))) return;
      if (!(ok = mbar_wait(&bars->k_full[stage], ph, a.status, wait_limit<kTest>(a)))) return;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(acc * 128);
      const uint32_t q_lo = umma_desc_lo(smem_u32(tiles + kOffQ + qb * kQBytes));
      const uint32_t k_lo = umma_desc_lo(smem_u32(tiles + kOffK + stage * kKStageBytes));
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        // k-step kk reads 32 bytes at offset (kk & 3) * 32 of sub-tile kk >> 2: the address field moves by
        // that many 16-byte units (tiles are 1024-byte aligned, so nothing carries out of the field)
        const uint32_t off = (uint32_t)(((kk >> 2) * kSubTileBytes + (kk & 3) * 32) >> 4);
        const uint64_t qd = desc64(q_lo + off, kDescHi), kd = desc64(k_lo + off, kDescHi);
        if (kk < nk) {
          if (kk == 0) umma_step<0>(d_tmem, pass == 0 ? qd : kd, pass == 0 ? kd : qd, idesc);
          else umma_step<1>(d_tmem, pass == 0 ? qd : kd, pass == 0 ? kd : qd, idesc);
        }
      }
      // pass 2: D -= off / c, as one more k-step over the constant tile and the rows' offset extensions
      if (pass == 1) umma_step<1>(d_tmem, fold_desc, ext_desc, idesc);
      tc_commit(&bars->k_empty[stage]);
      tc_commit(&bars->acc_full[acc]);
    }
    tc_commit(&bars->q_empty[qb]);          // Q (and the extension) are free once the segment's products are done
    if (pass == 1) {
      tc_commit(&bars->ext_empty[slot]);
      ++pc;
    }
    ++sc;
  });
}

// One 32-key chunk of a row: fold it into the running pair (M, Z) with Z = sum of 2^{c w - M}.
// M is a shift, not necessarily the maximum: any value within 2^kShiftSlack of the largest logit seen
// keeps every term finite, so the exponentials of a chunk are taken against the shift the row already
// has, and their sum tells whether that was sound: below 2^kShiftSlack, no term outran the shift by more
// than the slack.  Only otherwise (or when the row has no shift yet) is the chunk's maximum looked for and
// the chunk redone against it.
constexpr float kShiftSlack = 64.f;
constexpr float kAcceptBelow = 18446744073709551616.f;   // 2^kShiftSlack

__device__ __forceinline__ void fold_chunk(const uint32_t* r, bool full, int j_first, int last, float c, float& M,
                                           float& Z) {
  float v[32];
#pragma unroll
  for (int t = 0; t < 32; ++t) v[t] = __uint_as_float(r[t]);
  if (!full) {
#pragma unroll
    for (int t = 0; t < 32; ++t)
      if (j_first + t > last) v[t] = -INFINITY;
  }
  if (M > -INFINITY) {
    const float neg = -M;
    const uint64_t c2 = pack2(c, c), neg2 = pack2(neg, neg);
    uint64_t za = pack2(0.f, 0.f), zb = pack2(0.f, 0.f);
#pragma unroll
    for (int t = 0; t < 32; t += 4) {
      float x0, x1, x2, x3;
      unpack2(fma2(pack2(v[t], v[t + 1]), c2, neg2), x0, x1);
      unpack2(fma2(pack2(v[t + 2], v[t + 3]), c2, neg2), x2, x3);
      za = add2(za, pack2(fast_exp2(x0), fast_exp2(x1)));
      zb = add2(zb, pack2(fast_exp2(x2), fast_exp2(x3)));
    }
    float z0, z1, z2, z3;
    unpack2(za, z0, z1);
    unpack2(zb, z2, z3);
    const float z = (z0 + z1) + (z2 + z3);
    if (z < kAcceptBelow) {                          // an overflow or a NaN fails this test too
      Z += z;
      return;
    }
  }
  float mx0 = fmaxf(v[0], v[1]), mx1 = fmaxf(v[2], v[3]);
#pragma unroll
  for (int t = 4; t < 32; t += 4) {
    mx0 = fmaxf(mx0, fmaxf(v[t], v[t + 1]));
    mx1 = fmaxf(mx1, fmaxf(v[t + 2], v[t + 3]));
  }
  const float mx = fmaxf(mx0, mx1) * c;
  if (mx > -INFINITY) {                              // first visible keys of the row, or the shift fell behind
    const float neg = -mx;
    const uint64_t c2 = pack2(c, c), neg2 = pack2(neg, neg);
    uint64_t za = pack2(0.f, 0.f), zb = pack2(0.f, 0.f);
#pragma unroll
    for (int t = 0; t < 32; t += 4) {
      float x0, x1, x2, x3;
      unpack2(fma2(pack2(v[t], v[t + 1]), c2, neg2), x0, x1);
      unpack2(fma2(pack2(v[t + 2], v[t + 3]), c2, neg2), x2, x3);
      za = add2(za, pack2(fast_exp2(x0), fast_exp2(x1)));
      zb = add2(zb, pack2(fast_exp2(x2), fast_exp2(x3)));
    }
    float z0, z1, z2, z3;
    unpack2(za, z0, z1);
    unpack2(zb, z2, z3);
    Z = (M > -INFINITY ? Z * fast_exp2(M - mx) : 0.f) + ((z0 + z1) + (z2 + z3));
    M = mx;
  }
}

// Thirty-two stacked rows of a key's column, rows [32 Q, 32 Q + 32): adds 2^{c D} of each.  The column
// indices are compile-time constants, so every c comes straight from the kernel's parameter bank as an operand
// of the multiply.  The accumulator goes back to the MMA thread as soon as the values are in registers.
template <int Q>
__device__ __forceinline__ float column_sum_fast(const TcArgs& a, uint32_t taddr, void* acc_empty) {
  uint32_t r[32];
  tmem_ld32_issue(taddr + 32 * Q, r);
  tmem_ld_wait(r);
  tc_fence_before();
  mbar_arrive(acc_empty);
  uint64_t za = pack2(0.f, 0.f), zb = pack2(0.f, 0.f);
#pragma unroll
  for (int t = 0; t < 32; t += 4) {
    za = add2(za, pack2(fast_exp2(__uint_as_float(r[t]) * a.cs[32 * Q + t]),
                        fast_exp2(__uint_as_float(r[t + 1]) * a.cs[32 * Q + t + 1])));
    zb = add2(zb, pack2(fast_exp2(__uint_as_float(r[t + 2]) * a.cs[32 * Q + t + 2]),
                        fast_exp2(__uint_as_float(r[t + 3]) * a.cs[32 * Q + t + 3])));
  }
  float z0, z1, z2, z3;
  unpack2(za, z0, z1);
  unpack2(zb, z2, z3);
  return (z0 + z1) + (z2 + z3);
}

// Softmax warps: sixteen warps in four 4-warp groups, all of them on every tile (the four accumulators are used
// in turn); group g takes a quarter of the accumulator's columns, reads it with one load and hands the
// accumulator back before its arithmetic.  Which thread adds what does not depend on the schedule.
//   pass 1: thread `s` of a group owns stacked row s over its 32 key columns; at the end of the run the
//           four groups' (shift, sum) pairs meet in shared memory and one group publishes the row's
//           partial, log2 of the sum, with one 4-byte store.
//   pass 2: thread `jl` owns key j0 + jl over its quarter of the stacked rows; three groups hand their partial
//           sums over through shared memory, the first adds the four in a fixed order and stores.
template <bool kTest>
__device__ __forceinline__ void softmax_group(const TcArgs& a, Shared* sh, uint32_t tmem_base, int g) {
  Barriers* bars = &sh->bars;
  const int s = threadIdx.x & 127, quarter = (threadIdx.x >> 5) & 3;
  const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
  int tc = 0, p1c = 0;   // tiles and pass-1 runs seen so far
  bool gone = false;   // a wait ran out: keep only the barriers
  for_each_segment<kTest>(a, sh, [&](int pass, int run, int idx) {
    const Run rn = run_info(a, run);
    const UnitInfo u = unit_info(a, rn.unit);
    if (pass == 0) {
      const int i = obs_row(a, u, s);
      const float c = sh->c[i < a.r ? i : 0];
      const int last = a.last[i < kMaxRows ? i : 0];        // last visible key of this row
      float M = -INFINITY, Z = 0.f;
      for (int t = 0; t < rn.cnt; ++t, ++tc) {
        if (gone) continue;
        const int acc = tc & 3, aph = (tc >> 2) & 1;
        if (!mbar_wait(&bars->acc_full[acc], aph, a.status, wait_limit<kTest>(a))) { gone = true; continue; }
        tc_fence_after();
        const int j0 = (rn.blk0 + t) * kKeyTile + 32 * g;
        const bool full = (rn.blk0 + t) * kKeyTile + kKeyTile - 1 <= a.min_last;   // no key of the tile is masked
        uint32_t ra[32];
        tmem_ld32_issue(lane_base + (uint32_t)(acc * 128 + 32 * g), ra);
        tmem_ld_wait(ra);
        tc_fence_before();
        mbar_arrive(&bars->acc_empty[acc]);                  // the accumulator is free for the next product
        fold_chunk(ra, full, j0, last, c, M, Z);
      }
      // All sixteen warps meet here once per run, also after a wait has run out, so that nobody is left
      // at the barrier.  Two slots: the others can be at most one run ahead of the publishing group's read.
      const int slot = p1c & 1;
      ++p1c;
      if (g != 0) sh->p1_part[slot][g - 1][s] = make_float2(M, Z);
      group_sync(5, 512);
      if (g == 0 && !gone) {
        float m = M;
#pragma unroll
        for (int w = 0; w < 3; ++w) m = fmaxf(m, sh->p1_part[slot][w][s].x);
        float z = Z > 0.f ? Z * fast_exp2(M - m) : 0.f;
#pragma unroll
        for (int w = 0; w < 3; ++w) {
          const float2 e = sh->p1_part[slot][w][s];
          if (e.y > 0.f) z += e.y * fast_exp2(e.x - m);
        }
        float L = z > 0.f ? m + log2f(z) : -INFINITY;
        if (L != L) L = INFINITY;                            // NaN inputs: never publish the 'not yet' pattern
        if (!(kTest && a.test_withhold && rn.unit == 0 && rn.rin == 0))
          st_partial(&a.partial[((size_t)rn.unit * a.rpu + rn.rin) * 128 + s], L);
      }
    } else {
      const int jl = s;
      const int k16 = u.npad / 16;
      const int c_lo = (k16 * g / 4) * 16, c_hi = (k16 * (g + 1) / 4) * 16;   // this group's accumulator columns
      const bool fast = a.r <= 128 && u.rows == 128;
      const float* cs = sh->cs2[u.rb & 1];
      const int* last_key = sh->vis_off[u.rb & 1];
      for (int t = 0; t < rn.cnt; ++t, ++tc) {
        const int buf = tc & 1, acc = tc & 3, aph = (tc >> 2) & 1;
        const int j0 = (rn.blk0 + t) * kKeyTile, j = j0 + jl;
        float sum = 0.f;
        if (!gone && !mbar_wait(&bars->acc_full[acc], aph, a.status, wait_limit<kTest>(a))) gone = true;
        if (!gone) {
          tc_fence_after();
          const bool full = j0 + kKeyTile - 1 <= a.min_last;
          const uint32_t taddr = lane_base + (uint32_t)(acc * 128);
          if (full && fast) {
            void* ae = &bars->acc_empty[acc];
            sum = g == 0 ? column_sum_fast<0>(a, taddr, ae) : g == 1 ? column_sum_fast<1>(a, taddr, ae)
                : g == 2 ? column_sum_fast<2>(a, taddr, ae) : column_sum_fast<3>(a, taddr, ae);
          } else {
            // The product wrote exactly npad (a multiple of 16) columns; those past `rows` belong to no row.
#pragma unroll 1
            for (int s0 = c_lo; s0 < c_hi; s0 += 16) {
              uint32_t v[16];
              tmem_ld16_issue(taddr + s0, v);
              tmem_ld_wait16(v);
#pragma unroll
              for (int t2 = 0; t2 < 16; ++t2) {
                const int sr = s0 + t2;
                const bool vis = sr < u.rows && (full || j <= last_key[sr]);
                if (vis) sum += fast_exp2(__uint_as_float(v[t2]) * cs[sr]);
              }
            }
            tc_fence_before();
            mbar_arrive(&bars->acc_empty[acc]);
          }
        }
        // The four groups meet here once per tile, also after a wait has run out.  Two slots: the others can be
        // at most one tile ahead of the storing group's read.
        if (g != 0) sh->p2_part[buf][g - 1][jl] = sum;
        group_sync(6, 512);
        if (g == 0 && !gone && j < a.n)
          a.s_raw[(size_t)rn.unit * a.n + j] = ((sum + sh->p2_part[buf][0][jl]) + sh->p2_part[buf][1][jl]) + sh->p2_part[buf][2][jl];
      }
    }
    if (g == 0 && s == 0) *(volatile int*)&sh->seg_done_soft = idx + 1;   // lets the scheduler publish on
  });
}

// One row's offset extension: -off / (2 c kFold) as three 16-bit parts, the first three of the row's
// sixteen elements, the same again in the second 16-byte half.
__device__ __forceinline__ void write_extension(char* ext, int row, float off, float c, int bf16, bool live) {
  uint32_t w0 = 0, w1 = 0;
  if (live) {
    float v = -(off / c) / (2.f * kFold);
    if (bf16) {
      const __nv_bfloat16 h1 = __float2bfloat16_rn(v);
      v -= __bfloat162float(h1);
      const __nv_bfloat16 h2 = __float2bfloat16_rn(v);
      v -= __bfloat162float(h2);
      const __nv_bfloat16 h3 = __float2bfloat16_rn(v);
      w0 = (uint32_t)__bfloat16_as_ushort(h1) | ((uint32_t)__bfloat16_as_ushort(h2) << 16);
      w1 = (uint32_t)__bfloat16_as_ushort(h3);
    } else {
      v = fminf(fmaxf(v, -60000.f), 60000.f);              // float16 has no room beyond; such logits are not scored
      const __half h1 = __float2half_rn(v);
      v -= __half2float(h1);
      const __half h2 = __float2half_rn(v);
      v -= __half2float(h2);
      const __half h3 = __float2half_rn(v);
      w0 = (uint32_t)__half_as_ushort(h1) | ((uint32_t)__half_as_ushort(h2) << 16);
      w1 = (uint32_t)__half_as_ushort(h3);
    }
  }
  uint4* dst = reinterpret_cast<uint4*>(ext + row * 32);
  dst[0] = make_uint4(w0, w1, 0u, 0u);
  dst[1] = make_uint4(w0, w1, 0u, 0u);
}

// Merge group (two warps, 64 threads).  For every pass-2 run the scheduler announces, in order and
// ahead of the MMA warp: thread `s` waits until the partials of rows 2s and 2s + 1 have arrived from all runs of the
// row block, merges them in run order into the rows' offsets and writes their offset extensions into
// shared memory.
template <bool kTest>
__device__ void merge_group(const TcArgs& a, Shared* sh, char* tiles, int s) {
  Barriers* bars = &sh->bars;
  for (int mc = 0;; ++mc) {
    const int run = mrg_get(sh, mc, a.status, wait_limit<kTest>(a));
    if (run == kSegEnd) return;
    const Run rn = run_info(a, run);
    const UnitInfo u = unit_info(a, rn.unit);
    const int slot = mc & 1;
    if (!mbar_wait(&bars->ext_empty[slot], ((mc >> 1) & 1) ^ 1, a.status, wait_limit<kTest>(a))) return;
    const float2* p = reinterpret_cast<const float2*>(a.partial + (size_t)rn.unit * a.rpu * 128) + s;
    float M0 = -INFINITY, Z0 = 0.f, M1 = -INFINITY, Z1 = 0.f;   // running shift and sum of 2^{L - shift}, per row
    for (int t0 = 0; t0 < a.rpu; t0 += 16) {              // 16 8-byte loads in flight per thread
      float2 e[16];
      const long long tstart = now_ns();
      for (;;) {
        int missing = -1;
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          e[t] = t0 + t < a.rpu ? ld_partial2(&p[(size_t)(t0 + t) * 64]) : make_float2(-INFINITY, -INFINITY);
          if (!(e[t].x == e[t].x) || !(e[t].y == e[t].y)) missing = t;   // NaN: not published yet
        }
        if (missing < 0) break;
        // wait for that one partial alone before looking at the batch again: sixteen loads per thread and try
        // from every CTA that is early would keep L2 busy for nothing
        bool timed_out = false;
        for (;;) {
          __nanosleep(400);
          const float2 x = ld_partial2(&p[(size_t)(t0 + missing) * 64]);
          if (x.x == x.x && x.y == x.y) break;
          if (now_ns() - tstart > wait_limit<kTest>(a)) { timed_out = true; break; }
        }
        if (timed_out) {
          // nothing more is delivered; the MMA warp's own wait then runs out too
          atomicExch(a.status, (int)AHAKV_ERR_TIMEOUT);
          return;
        }
      }
      float m0 = M0, m1 = M1;
#pragma unroll
      for (int t = 0; t < 16; ++t) { m0 = fmaxf(m0, e[t].x); m1 = fmaxf(m1, e[t].y); }
      if (m0 > -INFINITY) {
        float z = Z0 > 0.f ? Z0 * fast_exp2(M0 - m0) : 0.f;
#pragma unroll
        for (int t = 0; t < 16; ++t) z += fast_exp2(e[t].x - m0);   // 2^{-inf} = 0 for the padding
        Z0 = z; M0 = m0;
      }
      if (m1 > -INFINITY) {
        float z = Z1 > 0.f ? Z1 * fast_exp2(M1 - m1) : 0.f;
#pragma unroll
        for (int t = 0; t < 16; ++t) z += fast_exp2(e[t].y - m1);
        Z1 = z; M1 = m1;
      }
    }
    // 2^{c w - off} = softmax weight / G.  The MMA adds 2 kFold (h1 + h2 + h3) = -off / c to w.
    char* ext = tiles + kOffExt + slot * kExtBytes;
    const int r0 = 2 * s, r1 = 2 * s + 1;
    write_extension(ext, r0, M0 + log2f(Z0) + a.log2G, sh->c[obs_row(a, u, r0 < u.rows ? r0 : 0)], a.bf16, r0 < u.rows);
    write_extension(ext, r1, M1 + log2f(Z1) + a.log2G, sh->c[obs_row(a, u, r1 < u.rows ? r1 : 0)], a.bf16, r1 < u.rows);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads it through the async proxy
    mbar_arrive(&bars->ext_full[slot]);
    if (s == 0) *(volatile int*)&sh->mrg_done = mc + 1;
  }
}

template <bool kTest>
__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                const __grid_constant__ CUtensorMap vmap, const __grid_constant__ TcArgs a) {
  extern __shared__ char smem_raw[];
  char* tiles = reinterpret_cast<char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Shared* sh = reinterpret_cast<Shared*>(tiles + kSmemTiles);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {   // the copy engine's descriptors on their way while the CTA sets itself up
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&qmap)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&kmap)) : "memory");
    if (a.prior) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&vmap)) : "memory");
  }
  for (int t = threadIdx.x; t < kMaxRows; t += kThreads) sh->c[t] = a.c[t];
  for (int t = threadIdx.x; t < 128; t += kThreads) {
    sh->cs2[0][t] = a.r <= 128 ? a.c[t % a.r] : a.c[t];
    sh->cs2[1][t] = a.r <= 128 ? a.c[t % a.r] : a.c[128 + t];
    sh->vis_off[0][t] = a.last[a.r <= 128 ? t % a.r : t];
    sh->vis_off[1][t] = a.last[a.r <= 128 ? t % a.r : 128 + t];
  }
  {
    // every 16-byte chunk of the constant tile reads (kFold, kFold, kFold, 0, 0, 0, 0, 0); it meets the
    // three parts of a row's extension twice, once per 16-byte half of the row
    const uint32_t one = a.bf16 ? (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(kFold))
                                : (uint32_t)__half_as_ushort(__float2half_rn(kFold));
    uint4* f = reinterpret_cast<uint4*>(tiles + kOffExt + 2 * kExtBytes);
    for (int t = threadIdx.x; t < kExtBytes / 16; t += kThreads) f[t] = make_uint4(one | (one << 16), one, 0u, 0u);
  }
  // Q rows a TMA box never covers (row blocks with fewer than 128 rows) must read as zeros, not as
  // whatever the last kernel left: zero both Q buffers once, before any bulk copy is issued.
  {
    uint4* z = reinterpret_cast<uint4*>(tiles + kOffQ);
    for (int t = threadIdx.x; t < 2 * kQBytes / 16; t += kThreads) z[t] = make_uint4(0, 0, 0, 0);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x == 0) {
    Barriers* bars = &sh->bars;
    for (int p = 0; p < 2; ++p) {
      mbar_init(&bars->q_full[p], 1);
      mbar_init(&bars->q_empty[p], 1);
      mbar_init(&bars->ext_full[p], 64);
      mbar_init(&bars->ext_empty[p], 1);
    }
    for (int s = 0; s < kVStages; ++s) {
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 128);
    }
    for (int s = 0; s < kKStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 1);
    }
    for (int s = 0; s < 4; ++s) {
      mbar_init(&bars->acc_full[s], 1);
      mbar_init(&bars->acc_empty[s], 512);
    }
    sh->seg_pub = 0; sh->seg_done_soft = 0; sh->seg_done_v = a.prior ? 0 : 0x3fffffff;
    sh->mrg_pub = 0; sh->mrg_done = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // all 512 TMEM columns: four 128-column accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sh->tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_slot;

  if (warp == 0) {
    if (lane == 0) producer<kTest>(a, &qmap, &kmap, &vmap, sh, tiles);
  } else if (warp == 1) {
    if (lane == 0) mma_issuer<kTest>(a, sh, tiles, tmem_base);
  } else if (warp < 4) {
    merge_group<kTest>(a, sh, tiles, threadIdx.x & 63);
  } else if (warp < 20) {
    softmax_group<kTest>(a, sh, tmem_base, (warp - 4) >> 2);
  } else {
    if (a.prior) v_group<kTest>(a, sh, tiles);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

// ---- host ------------------------------------------------------------------------------------------------
}  // namespace

bool score_tc_available() { return encode_fn() != nullptr; }

// Test hooks (see ahakv_test_set_wait): the limit of the kernel's bounded waits, and a planted fault.  While either
// is set, launches go to the test instantiation of the kernel.
static std::atomic<long long> g_test_wait_ns{0};
static std::atomic<int> g_test_withhold{0};
void score_tc_test_hooks(long long wait_ns, int withhold) {
  g_test_wait_ns.store(wait_ns > 0 ? wait_ns : 0);
  g_test_withhold.store(withhold);
}

ahakv_status launch_score_tc(const Plan& pl, const void* q, const void* k, const void* v, float* s_raw, float* nu,
                             float2* partial_ws, int* counters, int* status, cudaStream_t st) {
  // once per device: its SM count, and leave to use more than 48 KB of dynamic shared memory
  constexpr int kMaxDevices = 64;
  static int sm_count[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AHAKV_ERR_CUDA;
  if (sm_count[dev] == 0) {
    int count = 0;
    if (cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || count <= 0 ||
        cudaFuncSetAttribute(score_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(score_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
      return AHAKV_ERR_CUDA;
    sm_count[dev] = count;
  }
  const int n_sm = sm_count[dev];
  const int units = pl.B * pl.Hkv * pl.n_rb;
  TcArgs a;
  a.n = pl.n; a.r = pl.r; a.G = pl.G; a.Hkv = pl.Hkv; a.n_rb = pl.n_rb; a.hb = pl.heads_per_rb;
  a.n_blk = (pl.n_eff + kKeyTile - 1) / kKeyTile;   // tiles beyond are seen by no row
  a.D = pl.d;
  for (int i = 0; i < kMaxRows; ++i) a.last[i] = pl.last[i];
  a.min_last = pl.last[0];
  // Runs of 8 tiles; shorter ones (4, 2, 1) only as far as it takes to give three SMs in four a run.  Every run
  // boundary drains the pipeline, which costs more than a few idle SMs on a small problem.
  a.CH = 8;
  while (a.CH > 1 && (long long)units * ((a.n_blk + a.CH - 1) / a.CH) * 4 < (long long)n_sm * 3) a.CH >>= 1;
  a.rpu = (a.n_blk + a.CH - 1) / a.CH;
  a.n_runs = units * a.rpu;
  const int grid = a.n_runs < n_sm ? a.n_runs : n_sm;
  a.bf16 = pl.dtype == AHAKV_BF16;
  a.prior = (pl.flags & AHAKV_FLAG_VALUE_PRIOR) != 0 && v != nullptr && nu != nullptr;
  a.log2G = pl.group_max ? 0.f : log2f((float)pl.G);   // pooling by maximum keeps each head's own score
  for (int i = 0; i < kMaxRows; ++i) a.c[i] = pl.rows.c[i];
  for (int t = 0; t < 128; ++t) a.cs[t] = pl.r <= 128 ? pl.rows.c[t % pl.r] : 0.f;
  a.partial = reinterpret_cast<float*>(partial_ws); a.s_raw = s_raw; a.nu = nu;
  a.ctr = counters;
  a.status = status;
  a.test_wait_ns = g_test_wait_ns.load();
  a.test_withhold = g_test_withhold.load();
  const bool test = a.test_wait_ns > 0 || a.test_withhold != 0;
  if (a.test_wait_ns <= 0) a.test_wait_ns = kWaitLimitNs;

  CUtensorMap qmap, kmap, vmap;
  const int q_box_rows = pl.r <= 128 ? pl.r : 128, q_box_heads = pl.r <= 128 ? pl.heads_per_rb : 1;
  if (!make_map(&qmap, q, a.bf16, pl.d, pl.r, pl.Hq, pl.B, pl.qs, pl.es, q_box_rows, q_box_heads) ||
      !make_map(&kmap, k, a.bf16, pl.d, pl.n, pl.Hkv, pl.B, pl.ks, pl.es, kKeyTile, 1))
    return AHAKV_ERR_CUDA;
  if (a.prior) {
    if (!make_map(&vmap, v, a.bf16, pl.d, pl.n, pl.Hkv, pl.B, pl.vs, pl.es, kVRows, 1)) return AHAKV_ERR_CUDA;
  } else {
    vmap = kmap;   // never used
  }

  // every partial starts as NaN: "not published yet"
  if (cudaMemsetAsync(a.partial, 0xff, (size_t)a.n_runs * 128 * sizeof(float), st) != cudaSuccess) return AHAKV_ERR_CUDA;
  void* args[] = {&qmap, &kmap, &vmap, &a};
  const void* kernel = test ? (const void*)score_tc_kernel<true> : (const void*)score_tc_kernel<false>;
  const cudaError_t e = cudaLaunchCooperativeKernel(kernel, dim3(grid), dim3(kThreads), args, (size_t)kSmemBytes, st);
  count_launch();
  if (e != cudaSuccess) return AHAKV_ERR_CUDA;
  return cuda_ok(cudaGetLastError());
}

}  // namespace ahakv
