// Tensor-core scoring with the softmax numerators resident in tensor memory: every key tile is
// fetched once, multiplied once and exponentiated once.
//
// The accumulated SG-softmax score (Eq. 1, 5, 9) needs each observation row's normaliser over ALL
// keys before any normalised weight can be added into a key's score.  Here a 128-row x 128-key tile
// of logits D = Q . K^T (tcgen05.mma kind::f16, FP32 accumulator in tensor memory, rows on lanes)
// is turned in place into e_ij = 2^{c_i w_ij - m_i}, m_i the row's maximum over the tile, and STAYS
// in tensor memory while the row sums of all tiles of the row block meet:
//
//   phase A (per tile):  row maximum, e written back over the logits, log2 of the row's sum
//                        published as one 4-byte partial per row and tile;
//   merge (per row block): a warp somewhere on the GPU adds the partials of eight rows over all tiles,
//                        in tile order, and publishes the rows' log2 normalisers L_i;
//   phase B (per tile):  e_ij 2^{m_i - L_i} / G is summed over the 128 rows (lanes) by a fixed butterfly
//                        of warp shuffles and a shared-memory step across the four warps: the tile's
//                        column sums, stored as the raw score of its keys.
//
// Tensor memory holds four such tiles per SM (512 columns), so the tiles of about 2.3 heads of 32K
// tokens are in flight over the GPU at any time.  Tiles go to CTAs round-robin (tile T to CTA
// T mod grid), so the tiles of a row block finish phase A on all SMs at about the same time.  Each
// of the four accumulator slots belongs to one group of four softmax warps, which takes its tile
// through phase A, waits for the normalisers, and takes it through phase B; the four groups are
// out of step with one another, so the waits of one are the work of the others, and no barrier
// spans more than one group.  The value rows of each tile stream through a ring of their own and are
// squared and added by four warps (Section 4.3): nu_j = |V_j|^2 costs no second sweep of HBM.
//
// No deadlock: the launch is cooperative (all CTAs are resident), a slot is reused four positions
// later, i.e. 4 x grid tiles later, and launch_score_res takes only problems with at most 3 x grid
// tiles per row block, so the tile that frees a slot always belongs to an earlier row block than the
// tile that needs it, and row blocks are merged in order.  Every wait is bounded in time; on expiry the
// kernel records AHAKV_ERR_TIMEOUT in the status word and winds down.
//
// Results do not depend on timing: partials are merged in tile order by a fixed tree, the butterfly
// and the cross-warp sums have a fixed order, and nothing is accumulated with atomics.
#include <cuda.h>

#include "ahakv_internal.cuh"
#include "tc_common.cuh"

namespace ahakv {
namespace {

using namespace tc;

constexpr int kKStages = 3;                // K-tile ring depth
constexpr int kSubTileBytes = 128 * 128;   // 128 rows x 64 16-bit elements, 128-byte swizzled
constexpr int kVRows = 64;                 // value rows per V-ring stage
constexpr int kVStages = 2;
constexpr int kVSubBytes = kVRows * 128;
constexpr int kSlots = 4;                  // accumulator slots = softmax groups
constexpr int kThreads = 768;              // TMA warp, MMA warp, 2 merge warps, 16 softmax warps, 4 value-norm warps
constexpr int kMergeRows = 8;              // rows a merge task covers
constexpr int kTasksPerUnit = 128 / kMergeRows;

struct ResArgs {
  int n, r, G, Hkv, n_rb, hb, n_blk, D;
  int n_units;
  long long n_tiles;     // n_units * n_blk
  int bf16, prior;
  float log2G;
  float c[kMaxRows];     // lambda_i log2(e) per observation row
  float* partial;        // [unit][tile][128]: log2 of a row's sum of 2^{c w} over the tile's keys
  float* lfin;           // [unit][128]: log2 of the row's sum over all keys
  float* s_raw;          // [unit][n]
  float* nu;             // [B * Hkv][n]
  int* status;
};

struct __align__(8) Barriers {
  unsigned long long q_full[2], q_empty[2];
  unsigned long long k_full[kKStages], k_empty[kKStages];
  unsigned long long v_full[kVStages], v_empty[kVStages];
  unsigned long long acc_full[kSlots], acc_empty[kSlots];
};

struct Shared {
  Barriers bars;
  uint32_t tmem_slot;
  int abort;                               // a wait ran out somewhere in this CTA: everybody winds down
  float c[kMaxRows];
  float red[2][kSlots][4][128];            // phase B: column sums of each warp of a group, two tiles deep
};

constexpr int kQBytes = 2 * kSubTileBytes;
constexpr int kKStageBytes = 2 * kSubTileBytes;
constexpr int kVStageBytes = 2 * kVSubBytes;
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + 2 * kQBytes;
constexpr int kOffV = kOffK + kKStages * kKStageBytes;
constexpr int kSmemTiles = kOffV + kVStages * kVStageBytes;   // 192 KiB
constexpr int kSharedBytes = (sizeof(Shared) + 255) / 256 * 256;
constexpr int kSmemBytes = kSmemTiles + 1024 /*alignment slack*/ + kSharedBytes;
static_assert(kSmemBytes <= 227 * 1024, "shared memory budget");

struct UnitInfo {
  int unit, bh, rb, b, h, rows;
};
__device__ __forceinline__ UnitInfo unit_info(const ResArgs& a, int unit) {
  UnitInfo u;
  u.unit = unit;
  u.bh = unit / a.n_rb;
  u.rb = unit % a.n_rb;
  u.b = u.bh / a.Hkv;
  u.h = u.bh % a.Hkv;
  // r <= 128: hb query heads a block (fewer in the last block of a KV head when hb does not divide G; the box
  // still brings hb heads' rows, and no result depends on those past `rows`); r > 128: one head over two blocks
  u.rows = a.r <= 128 ? min(a.hb, a.G - u.rb * a.hb) * a.r : min(128, a.r - u.rb * 128);
  return u;
}
// Observation row index (0 .. r-1) of stacked row s of a row block.
__device__ __forceinline__ int obs_row(const ResArgs& a, const UnitInfo& u, int s) {
  return a.r <= 128 ? s % a.r : u.rb * 128 + s;
}

__device__ __forceinline__ bool aborted(Shared* sh) { return *(volatile int*)&sh->abort != 0; }
__device__ __forceinline__ void give_up(const ResArgs& a, Shared* sh) {
  atomicExch(a.status, (int)AHAKV_ERR_TIMEOUT);
  *(volatile int*)&sh->abort = 1;
}

// ---- roles --------------------------------------------------------------------------------------------
// TMA producer (one thread).  Walks this CTA's tiles in order and feeds two independent streams,
// whichever has a free slot: Q (when the row block changes) and K tiles, and the value rows of the tiles of
// each KV head's first row block.
__device__ void producer(const ResArgs& a, const CUtensorMap* qmap, const CUtensorMap* kmap, const CUtensorMap* vmap,
                         Shared* sh, char* tiles) {
  Barriers* bars = &sh->bars;
  const int n_sub = a.D / 64;
  const int q_rows = a.r <= 128 ? a.hb * a.r : 128;
  const int q_bytes = n_sub * q_rows * 128, k_bytes = n_sub * kSubTileBytes;
  const unsigned long long once = policy_evict_first();
  const long long grid = gridDim.x;

  long long kT = blockIdx.x;     // K stream: next tile
  int k_unit = -1, tc = 0, sc = -1;
  bool q_pending = false;
  long long vT = blockIdx.x;     // V stream: next tile, and the half of it to fetch
  int vt = 0, vc = 0;
  bool v_on = a.prior != 0;

  long long idle_since = -1;
  int idle_spins = 0;
  while (kT < a.n_tiles || (v_on && vT < a.n_tiles)) {
    if (aborted(sh)) break;
    bool progress = false;
    if (kT < a.n_tiles) {
      const int unit = (int)(kT / a.n_blk), t = (int)(kT % a.n_blk);
      if (unit != k_unit && !q_pending) { q_pending = true; ++sc; }
      const UnitInfo u = unit_info(a, unit);
      if (q_pending) {
        const int qb = sc & 1;
        if (mbar_test(&bars->q_empty[qb], ((sc >> 1) & 1) ^ 1)) {
          char* q_smem = tiles + kOffQ + qb * kQBytes;
          mbar_expect_tx(&bars->q_full[qb], q_bytes);
          for (int s = 0; s < n_sub; ++s) {
            if (a.r <= 128) tma_load_4d(q_smem + s * kSubTileBytes, qmap, &bars->q_full[qb], s * 64, 0, u.h * a.G + u.rb * a.hb, u.b);
            else tma_load_4d(q_smem + s * kSubTileBytes, qmap, &bars->q_full[qb], s * 64, u.rb * 128, u.h, u.b);
          }
          q_pending = false;
          k_unit = unit;
          progress = true;
        }
      } else {
        const int stage = tc % kKStages, ph = (tc / kKStages) & 1;
        if (mbar_test(&bars->k_empty[stage], ph ^ 1)) {
          mbar_expect_tx(&bars->k_full[stage], k_bytes);
          char* dst = tiles + kOffK + stage * kKStageBytes;
          // a key tile is read once per row block of its KV head; after the last one L2 may drop it first
          for (int s = 0; s < n_sub; ++s) {
            if (u.rb + 1 < a.n_rb) tma_load_4d(dst + s * kSubTileBytes, kmap, &bars->k_full[stage], s * 64, t * kKeyTile, u.h, u.b);
            else tma_load_4d_hint(dst + s * kSubTileBytes, kmap, &bars->k_full[stage], s * 64, t * kKeyTile, u.h, u.b, once);
          }
          ++tc;
          kT += grid;
          progress = true;
        }
      }
    }
    if (v_on && vT < a.n_tiles) {
      const int unit = (int)(vT / a.n_blk), t = (int)(vT % a.n_blk);
      const UnitInfo u = unit_info(a, unit);
      if (u.rb != 0) {
        vT += grid;
        progress = true;
      } else {
        const int vs = vc % kVStages;
        if (mbar_test(&bars->v_empty[vs], ((vc / kVStages) & 1) ^ 1)) {
          mbar_expect_tx(&bars->v_full[vs], n_sub * kVSubBytes);
          char* dst = tiles + kOffV + vs * kVStageBytes;
          for (int s = 0; s < n_sub; ++s)
            tma_load_4d_hint(dst + s * kVSubBytes, vmap, &bars->v_full[vs], s * 64, t * kKeyTile + vt * kVRows, u.h, u.b, once);
          ++vc;
          if (++vt == kKeyTile / kVRows) { vt = 0; vT += grid; }
          progress = true;
        }
      }
    }
    if (progress) {
      idle_since = -1;
      idle_spins = 0;
    } else if ((++idle_spins & 1023) == 0) {               // the clock is slow to read: look at it rarely
      const long long now = now_ns();
      if (idle_since < 0) idle_since = now;
      else if (now - idle_since > kWaitLimitNs) {
        give_up(a, sh);
        break;
      }
    }
  }
  if (aborted(sh)) {
    // wind down: give copies already in flight a bounded time (1 ms) to land before the CTA exits
    const long long t0 = now_ns();
    while (now_ns() - t0 < 1000000) __nanosleep(1000);
  }
}

// Value-norm group (four warps, 128 threads): two adjacent lanes share a row of each 64-row stage of the
// V ring (one half of its 16-byte chunks each, in an order that keeps them on different banks), square
// and add in FP32 and meet by shuffle: nu_j = |V_j|^2.
__device__ void v_group(const ResArgs& a, Shared* sh, char* tiles) {
  Barriers* bars = &sh->bars;
  const int row = (threadIdx.x & 127) >> 1, sub = threadIdx.x & 1;
  int ci = 0;
  for (long long T = blockIdx.x; T < a.n_tiles; T += gridDim.x) {
    const int unit = (int)(T / a.n_blk), t = (int)(T % a.n_blk);
    const UnitInfo u = unit_info(a, unit);
    if (u.rb != 0) continue;
    for (int vt = 0; vt < kKeyTile / kVRows; ++vt, ++ci) {
      const int vs = ci % kVStages;
      if (aborted(sh)) return;
      if (!mbar_wait(&bars->v_full[vs], (ci / kVStages) & 1, a.status)) { give_up(a, sh); return; }
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
      const int j = t * kKeyTile + vt * kVRows + row;
      if (sub == 0 && j < a.n) a.nu[(size_t)u.bh * a.n + j] = sq;
    }
  }
}

// MMA issuer (one thread): D[rows x keys] = Q K^T for this CTA's tiles in order, slot = position mod 4.
__device__ void mma_issuer(const ResArgs& a, Shared* sh, char* tiles, uint32_t tmem_base) {
  Barriers* bars = &sh->bars;
  const uint32_t idesc = umma_idesc(128, 128, a.bf16);
  const int nk = a.D / 16;
  int pos = 0, sc = -1, cur_unit = -1;
  for (long long T = blockIdx.x; T < a.n_tiles; T += gridDim.x, ++pos) {
    if (aborted(sh)) return;
    const int unit = (int)(T / a.n_blk);
    if (unit != cur_unit) {
      ++sc;
      cur_unit = unit;
      if (!mbar_wait(&bars->q_full[sc & 1], (sc >> 1) & 1, a.status)) { give_up(a, sh); return; }
    }
    const int qb = sc & 1;
    const int stage = pos % kKStages, ph = (pos / kKStages) & 1;
    const int slot = pos & (kSlots - 1), aph = (pos / kSlots) & 1;
    if (!mbar_wait(&bars->acc_empty[slot], aph ^ 1, a.status)) { give_up(a, sh); return; }
    if (!mbar_wait(&bars->k_full[stage], ph, a.status)) { give_up(a, sh); return; }
    tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)(slot * 128);
    const uint32_t q_lo = umma_desc_lo(smem_u32(tiles + kOffQ + qb * kQBytes));
    const uint32_t k_lo = umma_desc_lo(smem_u32(tiles + kOffK + stage * kKStageBytes));
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      // k-step kk reads 32 bytes at offset (kk & 3) * 32 of sub-tile kk >> 2: the address field moves by
      // that many 16-byte units (tiles are 1024-byte aligned, so nothing carries out of the field)
      const uint32_t off = (uint32_t)(((kk >> 2) * kSubTileBytes + (kk & 3) * 32) >> 4);
      const uint64_t qd = desc64(q_lo + off, kDescHi), kd = desc64(k_lo + off, kDescHi);
      if (kk < nk) {
        if (kk == 0) umma_step<0>(d_tmem, qd, kd, idesc);
        else umma_step<1>(d_tmem, qd, kd, idesc);
      }
    }
    tc_commit(&bars->k_empty[stage]);
    tc_commit(&bars->acc_full[slot]);
    const long long Tn = T + gridDim.x;
    if (Tn >= a.n_tiles || (int)(Tn / a.n_blk) != unit) tc_commit(&bars->q_empty[qb]);   // last tile of the row block here
  }
}

// Sum over the 32 lanes of a warp of each of 32 values: on return lane l holds the sum of v[l] over the lanes.
// A butterfly with a fixed order of additions: half of the values go to the partner lane at each step.
__device__ __forceinline__ float lane_transpose_sum(const float* v, int lane) {
  float w16[16], w8[8], w4[4], w2[2];
  {
    const bool up = (lane & 16) != 0;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const float send = up ? v[k] : v[k + 16], keep = up ? v[k + 16] : v[k];
      w16[k] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
  }
  {
    const bool up = (lane & 8) != 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float send = up ? w16[k] : w16[k + 8], keep = up ? w16[k + 8] : w16[k];
      w8[k] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
  }
  {
    const bool up = (lane & 4) != 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float send = up ? w8[k] : w8[k + 4], keep = up ? w8[k + 4] : w8[k];
      w4[k] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
  }
  {
    const bool up = (lane & 2) != 0;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const float send = up ? w4[k] : w4[k + 2], keep = up ? w4[k + 2] : w4[k];
      w2[k] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
  }
  const bool up = (lane & 1) != 0;
  const float send = up ? w2[0] : w2[1], keep = up ? w2[1] : w2[0];
  return keep + __shfl_xor_sync(0xffffffffu, send, 1);
}

// A published float, straight from L2 (other CTAs write it while this one polls); NaN = not yet there.
__device__ __forceinline__ float ld_published(const float* p) {
  float v;
  asm volatile("ld.relaxed.gpu.global.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
  return v;
}

// Softmax group g (four warps, 128 threads: thread s owns stacked row s = TMEM lane s) owns accumulator slot g,
// i.e. every fourth tile of this CTA, and takes each through phase A, the wait for the normalisers, and phase B.
__device__ void softmax_group(const ResArgs& a, Shared* sh, uint32_t tmem_base, int g) {
  Barriers* bars = &sh->bars;
  const int s = threadIdx.x & 127, lane = threadIdx.x & 31, quarter = (threadIdx.x >> 5) & 3;
  const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(g * 128);
  bool gone = false;           // a wait ran out: keep only the barriers
  int it = 0;
  for (long long T = blockIdx.x + (long long)g * gridDim.x; T < a.n_tiles; T += (long long)kSlots * gridDim.x, ++it) {
    const int unit = (int)(T / a.n_blk), t = (int)(T % a.n_blk);
    const UnitInfo u = unit_info(a, unit);
    const bool live = s < u.rows;
    const int i = obs_row(a, u, live ? s : 0);
    const float c = sh->c[i];
    const int j0 = t * kKeyTile;
    const int last = a.n - a.r + i;                            // last key this row may see
    const bool full = j0 + kKeyTile - 1 <= a.n - a.r;          // no key of the tile is masked for any row
    float colsum[4] = {0.f, 0.f, 0.f, 0.f};
    // A warp goes on together or not at all (the tensor-memory loads and stores below are warp-wide), so every
    // decision to give up is put to the vote of the whole warp.
    if (!gone && aborted(sh)) gone = true;
    if (!gone && !mbar_wait(&bars->acc_full[g], it & 1, a.status)) { give_up(a, sh); gone = true; }
    gone = __any_sync(0xffffffffu, gone);
    float m = 0.f, Lr = 0.f;
    bool any = false;
    if (!gone) {
      tc_fence_after();
      // ---- phase A, first sweep: the row's largest logit of the tile ----
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tmem_ld32_issue(taddr + 32 * ch, r);
        tmem_ld_wait(r);
        if (full) {
#pragma unroll
          for (int x = 0; x < 32; x += 2) {
            mx0 = fmaxf(mx0, __uint_as_float(r[x]));
            mx1 = fmaxf(mx1, __uint_as_float(r[x + 1]));
          }
        } else {
#pragma unroll
          for (int x = 0; x < 32; ++x)
            if (j0 + 32 * ch + x <= last) mx0 = fmaxf(mx0, __uint_as_float(r[x]));
        }
      }
      const float mx = fmaxf(mx0, mx1);
      any = mx > -INFINITY;                                    // the row sees at least one key of the tile
      m = any ? mx * c : 0.f;
      // ---- second sweep: e = 2^{c w - m} over the logits, and the row's sum ----
      uint64_t za = pack2(0.f, 0.f), zb = pack2(0.f, 0.f);
      const uint64_t c2 = pack2(c, c), neg2 = pack2(-m, -m);
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tmem_ld32_issue(taddr + 32 * ch, r);
        tmem_ld_wait(r);
#pragma unroll
        for (int x = 0; x < 32; x += 4) {
          float x0, x1, x2, x3;
          unpack2(fma2(pack2(__uint_as_float(r[x]), __uint_as_float(r[x + 1])), c2, neg2), x0, x1);
          unpack2(fma2(pack2(__uint_as_float(r[x + 2]), __uint_as_float(r[x + 3])), c2, neg2), x2, x3);
          float e0 = fast_exp2(x0), e1 = fast_exp2(x1), e2 = fast_exp2(x2), e3 = fast_exp2(x3);
          if (!full) {
            const int j = j0 + 32 * ch + x;
            if (j > last) e0 = 0.f;
            if (j + 1 > last) e1 = 0.f;
            if (j + 2 > last) e2 = 0.f;
            if (j + 3 > last) e3 = 0.f;
          }
          za = add2(za, pack2(e0, e1));
          zb = add2(zb, pack2(e2, e3));
          r[x] = __float_as_uint(e0); r[x + 1] = __float_as_uint(e1);
          r[x + 2] = __float_as_uint(e2); r[x + 3] = __float_as_uint(e3);
        }
        tmem_st32(taddr + 32 * ch, r);
      }
      tmem_st_wait();
      float z0, z1, z2, z3;
      unpack2(za, z0, z1);
      unpack2(zb, z2, z3);
      const float Z = (z0 + z1) + (z2 + z3);
      float L = (any && Z > 0.f) ? m + log2f(Z) : -INFINITY;
      if (L != L) L = INFINITY;                                // NaN inputs: never publish the 'not yet' pattern
      st_partial(&a.partial[((size_t)unit * a.n_blk + t) * 128 + s], L);

      // ---- the row's normaliser over all keys, from whoever merges this row block ----
      Lr = ld_published(&a.lfin[(size_t)unit * 128 + s]);
      if (Lr != Lr) {
        long long t0 = -1;
        for (int spins = 0;; ++spins) {
          __nanosleep(100);
          Lr = ld_published(&a.lfin[(size_t)unit * 128 + s]);
          if (Lr == Lr) break;
          if ((spins & 255) != 255) continue;                  // the clock is slow to read
          if (aborted(sh)) break;
          if (t0 < 0) t0 = now_ns();
          else if (now_ns() - t0 > kWaitLimitNs) { give_up(a, sh); break; }
        }
      }
      if (Lr != Lr) gone = true;
    }
    gone = __any_sync(0xffffffffu, gone);
    if (!gone) {
      // ---- phase B: the tile's column sums of e 2^{m - L} / G over this warp's 32 rows ----
      const float f = (live && any) ? fast_exp2(m - Lr - a.log2G) : 0.f;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tmem_ld32_issue(taddr + 32 * ch, r);
        tmem_ld_wait(r);
        float v[32];
#pragma unroll
        for (int x = 0; x < 32; ++x) v[x] = f > 0.f ? __uint_as_float(r[x]) * f : 0.f;
        colsum[ch] = lane_transpose_sum(v, lane);
      }
      tc_fence_before();
      mbar_arrive(&bars->acc_empty[g]);                        // the slot is free for the product four tiles on
    }
    // The four warps of the group meet here once per tile, also after a wait has run out.  Two buffers: the
    // others can be at most one tile ahead of the slowest thread's reads.
    float* red = &sh->red[it & 1][g][0][0];
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) red[quarter * 128 + 32 * ch + lane] = colsum[ch];
    group_sync(8 + g, 128);
    const int j = j0 + s;
    if (!gone && j < a.n) a.s_raw[(size_t)unit * a.n + j] = ((red[s] + red[128 + s]) + red[256 + s]) + red[384 + s];
  }
}

// Merge warps (two per CTA).  A task = eight rows of one row block: add, in tile order, the partials of all tiles
// into the rows' log2 normalisers.  Tasks are dealt round-robin over all merge warps of the grid and each
// warp takes its own in row-block order.  Lane = (row pair, tile stripe): four row pairs, eight stripes.
__device__ void merge_warp(const ResArgs& a, Shared* sh, int mw) {
  const int lane = threadIdx.x & 31, rp = lane & 3, stripe = lane >> 2;
  const long long n_tasks = (long long)a.n_units * kTasksPerUnit, warps = 2LL * gridDim.x;
  for (long long task = 2LL * blockIdx.x + mw; task < n_tasks; task += warps) {
    const int unit = (int)(task / kTasksPerUnit), slice = (int)(task % kTasksPerUnit);
    const int row0 = slice * kMergeRows + 2 * rp;
    const float2* p = reinterpret_cast<const float2*>(a.partial + (size_t)unit * a.n_blk * 128 + row0);
    float M0 = -INFINITY, Z0 = 0.f, M1 = -INFINITY, Z1 = 0.f;   // running shift and sum of 2^{L - shift}, per row
    bool failed = false;
    for (int t0 = 0; t0 < a.n_blk && !failed; t0 += 8 * 16) {    // 16 8-byte loads in flight per lane
      float2 e[16];
      const long long tstart = now_ns();
      for (;;) {
        int missing = -1;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const int t = t0 + stripe + 8 * k;
          e[k] = t < a.n_blk ? ld_partial2(&p[(size_t)t * 64]) : make_float2(-INFINITY, -INFINITY);
          if (!(e[k].x == e[k].x) || !(e[k].y == e[k].y)) missing = k;   // NaN: not published yet
        }
        if (missing < 0) break;
        // wait for that one partial alone before looking at the batch again
        for (;;) {
          __nanosleep(400);
          const float2 x = ld_partial2(&p[(size_t)(t0 + stripe + 8 * missing) * 64]);
          if (x.x == x.x && x.y == x.y) break;
          if (aborted(sh) || now_ns() - tstart > kWaitLimitNs) { failed = true; break; }
        }
        if (failed) break;
      }
      if (failed) break;
      float m0 = M0, m1 = M1;
#pragma unroll
      for (int k = 0; k < 16; ++k) { m0 = fmaxf(m0, e[k].x); m1 = fmaxf(m1, e[k].y); }
      if (m0 > -INFINITY) {
        float z = Z0 > 0.f ? Z0 * fast_exp2(M0 - m0) : 0.f;
#pragma unroll
        for (int k = 0; k < 16; ++k) z += fast_exp2(e[k].x - m0);   // 2^{-inf} = 0 for the padding
        Z0 = z; M0 = m0;
      }
      if (m1 > -INFINITY) {
        float z = Z1 > 0.f ? Z1 * fast_exp2(M1 - m1) : 0.f;
#pragma unroll
        for (int k = 0; k < 16; ++k) z += fast_exp2(e[k].y - m1);
        Z1 = z; M1 = m1;
      }
    }
    if (__any_sync(0xffffffffu, failed)) {
      if (!aborted(sh)) give_up(a, sh);
      return;
    }
    // the eight stripes of a row pair meet: lanes 4, 8, 16 apart, a fixed tree
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      const float pm0 = __shfl_xor_sync(0xffffffffu, M0, o), pz0 = __shfl_xor_sync(0xffffffffu, Z0, o);
      const float pm1 = __shfl_xor_sync(0xffffffffu, M1, o), pz1 = __shfl_xor_sync(0xffffffffu, Z1, o);
      const float n0 = fmaxf(M0, pm0), n1 = fmaxf(M1, pm1);
      // the lower lane's term first on both sides, so that partners hold the same bits
      const bool low = (lane & o) == 0;
      {
        const float mine = Z0 > 0.f ? Z0 * fast_exp2(M0 - n0) : 0.f, theirs = pz0 > 0.f ? pz0 * fast_exp2(pm0 - n0) : 0.f;
        Z0 = low ? mine + theirs : theirs + mine;
        M0 = n0;
      }
      {
        const float mine = Z1 > 0.f ? Z1 * fast_exp2(M1 - n1) : 0.f, theirs = pz1 > 0.f ? pz1 * fast_exp2(pm1 - n1) : 0.f;
        Z1 = low ? mine + theirs : theirs + mine;
        M1 = n1;
      }
    }
    if (stripe == 0) {
      float L0 = Z0 > 0.f ? M0 + log2f(Z0) : -INFINITY, L1 = Z1 > 0.f ? M1 + log2f(Z1) : -INFINITY;
      if (L0 != L0) L0 = INFINITY;
      if (L1 != L1) L1 = INFINITY;
      float* dst = a.lfin + (size_t)unit * 128 + row0;
      asm volatile("st.relaxed.gpu.global.v2.f32 [%0], {%1, %2};" ::"l"(dst), "f"(L0), "f"(L1) : "memory");
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
score_res_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                 const __grid_constant__ CUtensorMap vmap, const __grid_constant__ ResArgs a) {
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
    }
    for (int s = 0; s < kVStages; ++s) {
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 128);
    }
    for (int s = 0; s < kKStages; ++s) {
      mbar_init(&bars->k_full[s], 1);
      mbar_init(&bars->k_empty[s], 1);
    }
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&bars->acc_full[s], 1);
      mbar_init(&bars->acc_empty[s], 128);
    }
    sh->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // all 512 TMEM columns: four 128-column tiles
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sh->tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_slot;

  if (warp == 0) {
    if (lane == 0) producer(a, &qmap, &kmap, &vmap, sh, tiles);
  } else if (warp == 1) {
    if (lane == 0) mma_issuer(a, sh, tiles, tmem_base);
  } else if (warp < 4) {
    merge_warp(a, sh, warp - 2);
  } else if (warp < 20) {
    softmax_group(a, sh, tmem_base, (warp - 4) >> 2);
  } else {
    if (a.prior) v_group(a, sh, tiles);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

struct DeviceInfo {
  int sm_count;
};
// Once per device: its SM count, and leave to use more than 48 KB of dynamic shared memory.
ahakv_status device_info(DeviceInfo* out) {
  constexpr int kMaxDevices = 64;
  static int sm_count[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AHAKV_ERR_CUDA;
  if (sm_count[dev] == 0) {
    int count = 0;
    if (cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || count <= 0 ||
        cudaFuncSetAttribute(score_res_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
      return AHAKV_ERR_CUDA;
    sm_count[dev] = count;
  }
  out->sm_count = sm_count[dev];
  return AHAKV_OK;
}

}  // namespace

// Whether the resident kernel takes this problem: a row block may put at most three tiles on any one CTA (see the
// note on deadlock at the top), and tile indices must fit the kernel's arithmetic.
bool score_res_fits(const Plan& pl) {
  if (!pl.use_tc) return false;
  DeviceInfo di;
  if (device_info(&di) != AHAKV_OK) return false;
  const long long units = (long long)pl.B * pl.Hkv * pl.n_rb, tiles = units * pl.n_blk;
  const long long grid = tiles < di.sm_count ? tiles : di.sm_count;
  return pl.n_blk <= 3 * grid && units < (1LL << 24);
}

ahakv_status launch_score_res(const Plan& pl, const void* q, const void* k, const void* v, float* s_raw, float* nu,
                              float* partial, float* lfin, int* status, cudaStream_t st) {
  DeviceInfo di;
  ahakv_status rc = device_info(&di);
  if (rc) return rc;
  ResArgs a;
  a.n = pl.n; a.r = pl.r; a.G = pl.G; a.Hkv = pl.Hkv; a.n_rb = pl.n_rb; a.hb = pl.heads_per_rb;
  a.n_blk = pl.n_blk; a.D = pl.d;
  a.n_units = pl.B * pl.Hkv * pl.n_rb;
  a.n_tiles = (long long)a.n_units * pl.n_blk;
  const int grid = a.n_tiles < di.sm_count ? (int)a.n_tiles : di.sm_count;
  a.bf16 = pl.dtype == AHAKV_BF16;
  a.prior = (pl.flags & AHAKV_FLAG_VALUE_PRIOR) != 0 && v != nullptr && nu != nullptr;
  a.log2G = pl.group_max ? 0.f : log2f((float)pl.G);   // pooling by maximum keeps each head's own score
  for (int i = 0; i < kMaxRows; ++i) a.c[i] = pl.rows.c[i];
  a.partial = partial; a.lfin = lfin; a.s_raw = s_raw; a.nu = nu;
  a.status = status;

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

  // every partial and every normaliser starts as NaN: "not published yet"
  if (cudaMemsetAsync(partial, 0xff, (size_t)a.n_tiles * 128 * sizeof(float), st) != cudaSuccess ||
      cudaMemsetAsync(lfin, 0xff, (size_t)a.n_units * 128 * sizeof(float), st) != cudaSuccess)
    return AHAKV_ERR_CUDA;
  void* args[] = {&qmap, &kmap, &vmap, &a};
  const cudaError_t e = cudaLaunchCooperativeKernel((const void*)score_res_kernel, dim3(grid), dim3(kThreads), args,
                                                    (size_t)kSmemBytes, st);
  count_launch();
  if (e != cudaSuccess) return AHAKV_ERR_CUDA;
  return cuda_ok(cudaGetLastError());
}

}  // namespace ahakv
