// Tensor-core scoring for 16-bit inputs on sm_100a: one persistent kernel that
// computes the accumulated SG-softmax score (Eq. 1, 5, 9) of every KV head.
//
// Work unit: a "row block" = up to 128 stacked observation rows (query heads of
// one KV head x observation rows) against all n keys, cut into 128-key tiles.
// A normalised column sum needs each row's softmax statistics over ALL keys
// first, so every tile is visited twice, by two pipelines that live side by side
// in each CTA and share nothing but the SM:
//
//   pass 1 (rows on TMEM lanes):  D = Q . K^T   -> per-row (max, sum of 2^{c w - max})
//                                 of the tile, written as a partial; the CTA that
//                                 delivers a row block's last partial merges them
//                                 into one offset per row and raises the block's flag.
//   pass 2 (keys on TMEM lanes):  D = K . Q^T   -> each thread owns one key and adds
//                                 2^{c w - offset} over the rows: the column sum
//                                 needs no cross-thread traffic at all.
//
// Both products are tcgen05.mma kind::f16 with FP32 accumulators in TMEM, fed by
// TMA (128-byte swizzle) from the same K-major Q and K tiles, which serve as A or
// B operand alike.  Pass 2 trails pass 1 by a few row blocks, so its second read
// of K is served by L2 and HBM sees K once.
//
// Each pipeline has its own TMA warp, MMA warp and 4-warp softmax group; pass 1
// never waits on pass 2, so the flag waits of pass 2 cannot deadlock.  The kernel
// is launched cooperatively with at most one CTA per SM, which guarantees that
// the CTAs a flag depends on are running.  Every wait is bounded in time; on
// expiry the kernel records AHAKV_ERR_TIMEOUT in the status word and winds down.
#include <cuda.h>

#include "ahakv_internal.cuh"

namespace ahakv {
namespace {

constexpr int kStages = 2;                 // K-tile ring depth per pipeline
constexpr int kSubTileBytes = 128 * 128;   // 128 rows x 64 16-bit elements, 128-byte swizzled
constexpr int kThreads = 384;              // 4 service warps + two 4-warp softmax groups
constexpr long long kWaitLimitNs = 1000000000LL;   // 1 s

struct TcArgs {
  int n, r, G, Hkv, n_rb, hb, n_blk, D;
  int T;          // tiles = units * n_blk
  int CH;         // consecutive tiles per run
  int n_runs;
  int bf16;       // operand type of the products
  float log2G;
  float c[kMaxRows];
  float2* partial;   // [unit][blk][128]
  float* final_off;  // [unit][128]
  float* s_raw;      // [unit][n]
  int* cnt;          // [unit] partials delivered
  int* flag;         // [unit] rows whose offset is ready (128 = all)
  int* status;
};

// ---- shared memory layout --------------------------------------------------------------------
struct __align__(8) Barriers {
  unsigned long long q_full[2];            // [pipeline]
  unsigned long long k_full[2][kStages];
  unsigned long long k_empty[2][kStages];
  unsigned long long acc_full[2][2];
  unsigned long long acc_empty[2][2];
};

constexpr int kQBytes = 2 * kSubTileBytes;              // per pipeline, D <= 128
constexpr int kKRingBytes = kStages * 2 * kSubTileBytes;
constexpr int kSmemTiles = 2 * (kQBytes + kKRingBytes);  // 192 KiB
constexpr int kSmemBytes = kSmemTiles + 1024 /*alignment slack*/ + 4096 /*barriers, constants*/;

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ long long now_ns() {
  long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(void* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, int bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(void* bar, int parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and records the timeout) if the phase did not complete in time.
__device__ __forceinline__ bool mbar_wait(void* bar, int parity, int* status) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = now_ns();
  for (;;) {
#pragma unroll 1
    for (int t = 0; t < 64; ++t)
      if (mbar_try(bar, parity)) return true;
    if (now_ns() - t0 > kWaitLimitNs) {
      atomicExch(status, (int)AHAKV_ERR_TIMEOUT);
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, void* bar, int c0, int c1, int c2,
                                            int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(void* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// Shared-memory operand descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart, descriptor version 1 (sm_100).
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3ffff) >> 4);          // start address
  d |= (uint64_t)1 << 16;                               // leading byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset
  d |= (uint64_t)1 << 46;                               // version
  d |= (uint64_t)2 << 61;                               // SWIZZLE_128B
  return d;
}

// Instruction descriptor for kind::f16: FP32 accumulate, A and B both K-major and of one type.
__device__ __forceinline__ uint32_t umma_idesc(int M, int N, int bf16) {
  uint32_t d = 0;
  d |= 1u << 4;                         // D format F32
  d |= (uint32_t)(bf16 ? 1 : 0) << 7;   // A format
  d |= (uint32_t)(bf16 ? 1 : 0) << 10;  // B format
  d |= (uint32_t)(N >> 3) << 17;
  d |= (uint32_t)(M >> 4) << 24;
  return d;
}

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, int accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// 32 consecutive FP32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"      // one statement: no use of the registers can move above the wait
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int t = 0; t < 32; ++t) v[t] = __uint_as_float(r[t]);
}

// 16 consecutive FP32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int t = 0; t < 16; ++t) v[t] = __uint_as_float(r[t]);
}

__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// ---- the sequence of tiles one CTA walks (the same in every role) ----------------------------------
struct TileWalk {
  int run, t, t_end, T, CH, step;
  __device__ TileWalk(const TcArgs& a) : run(blockIdx.x), T(a.T), CH(a.CH), step(gridDim.x) { open(); }
  __device__ void open() {
    t = run * CH;
    t_end = min(t + CH, T);
  }
  __device__ bool valid() const { return t < T; }
  __device__ void next() {
    if (++t >= t_end) {
      run += step;
      open();
    }
  }
};

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
  u.rows = a.r <= 128 ? a.hb * a.r : min(128, a.r - u.rb * 128);
  u.npad = (u.rows + 15) & ~15;
  return u;
}
// Observation row index (0 .. r-1) of stacked row s of a row block.
__device__ __forceinline__ int obs_row(const TcArgs& a, const UnitInfo& u, int s) {
  return a.r <= 128 ? s % a.r : u.rb * 128 + s;
}

// ---- roles --------------------------------------------------------------------------------------------
// TMA producer of one pipeline.
__device__ void producer(const TcArgs& a, const CUtensorMap* qmap, const CUtensorMap* kmap, Barriers* bars, int pipe,
                         char* q_smem, char* k_ring) {
  const int n_sub = a.D / 64;
  const int q_rows = a.r <= 128 ? a.hb * a.r : 128;
  const int q_bytes = n_sub * q_rows * 128, k_bytes = n_sub * kSubTileBytes;
  int it = 0, prev_unit = -1, q_loads = 0;
  bool ok = true;
  for (TileWalk w(a); w.valid() && ok; w.next(), ++it) {
    const int unit = w.t / a.n_blk, blk = w.t % a.n_blk;
    const int stage = it % kStages, ph = (it / kStages) & 1;
    if (unit != prev_unit) {
      // the Q buffer is free once every product issued so far has completed
      if (it > 0) ok = mbar_wait(&bars->k_empty[pipe][(it - 1) % kStages], ((it - 1) / kStages) & 1, a.status);
      if (!ok) break;
      const UnitInfo u = unit_info(a, unit);
      mbar_expect_tx(&bars->q_full[pipe], q_bytes);
      for (int s = 0; s < n_sub; ++s) {
        if (a.r <= 128) tma_load_4d(q_smem + s * kSubTileBytes, qmap, &bars->q_full[pipe], s * 64, 0, u.h * a.G + u.rb * a.hb, u.b);
        else tma_load_4d(q_smem + s * kSubTileBytes, qmap, &bars->q_full[pipe], s * 64, u.rb * 128, u.h, u.b);
      }
      ++q_loads;
      prev_unit = unit;
    }
    ok = mbar_wait(&bars->k_empty[pipe][stage], ph ^ 1, a.status);
    if (!ok) break;
    const UnitInfo u = unit_info(a, unit);
    mbar_expect_tx(&bars->k_full[pipe][stage], k_bytes);
    for (int s = 0; s < n_sub; ++s)
      tma_load_4d(k_ring + (stage * 2 + s) * kSubTileBytes, kmap, &bars->k_full[pipe][stage], s * 64, blk * kKeyTile,
                  u.h, u.b);
  }
  if (!ok) {
    // wind down: give copies already in flight a bounded time (1 ms) to land before the CTA exits
    const long long t0 = now_ns();
    while (now_ns() - t0 < 1000000) __nanosleep(1000);
  }
  (void)q_loads;
}

// MMA issuer of one pipeline.  pipe 0: D[rows x keys] = Q K^T.  pipe 1: D[keys x rows] = K Q^T.
__device__ void mma_issuer(const TcArgs& a, Barriers* bars, int pipe, char* q_smem, char* k_ring, uint32_t tmem_base) {
  const int n_sub = a.D / 64;
  int it = 0, prev_unit = -1, q_loads = 0;
  uint32_t idesc = umma_idesc(128, 128, a.bf16);
  for (TileWalk w(a); w.valid(); w.next(), ++it) {
    const int unit = w.t / a.n_blk;
    const int stage = it % kStages, ph = (it / kStages) & 1, acc = it & 1, aph = (it >> 1) & 1;
    if (unit != prev_unit) {
      if (!mbar_wait(&bars->q_full[pipe], q_loads & 1, a.status)) return;
      ++q_loads;
      prev_unit = unit;
      if (pipe == 1) idesc = umma_idesc(128, unit_info(a, unit).npad, a.bf16);
    }
    if (!mbar_wait(&bars->acc_empty[pipe][acc], aph ^ 1, a.status)) return;
    if (!mbar_wait(&bars->k_full[pipe][stage], ph, a.status)) return;
    tc_fence_after();
    const uint32_t d_tmem = tmem_base + (uint32_t)((pipe * 2 + acc) * 128);
    for (int kk = 0; kk < a.D / 16; ++kk) {
      const int sub = kk >> 2, koff = (kk & 3) * 32;
      const uint64_t qd = umma_desc(smem_u32(q_smem + sub * kSubTileBytes) + koff);
      const uint64_t kd = umma_desc(smem_u32(k_ring + (stage * 2 + sub) * kSubTileBytes) + koff);
      if (pipe == 0) umma(d_tmem, qd, kd, idesc, kk > 0);
      else umma(d_tmem, kd, qd, idesc, kk > 0);
    }
    tc_commit(&bars->k_empty[pipe][stage]);
    tc_commit(&bars->acc_full[pipe][acc]);
  }
  (void)n_sub;
}

// Pass-1 softmax group: thread `s` owns stacked row s.
__device__ void row_stats_group(const TcArgs& a, Barriers* bars, uint32_t tmem_base, const float* c_smem, int* bcast) {
  const int s = threadIdx.x & 127, quarter = (threadIdx.x >> 5) & 3;
  int it = 0;
  bool dead = false;   // a wait ran out: stay in the group's barrier protocol, skip everything else
  for (TileWalk w(a); w.valid(); w.next(), ++it) {
    const int unit = w.t / a.n_blk, blk = w.t % a.n_blk;
    const UnitInfo u = unit_info(a, unit);
    const int acc = it & 1, aph = (it >> 1) & 1;
    if (!dead && !mbar_wait(&bars->acc_full[0][acc], aph, a.status)) dead = true;
    if (dead) {          // the three barriers of a live iteration, nothing else
      group_sync(1);
      if (s == 0) bcast[0] = -1;
      group_sync(1);
      group_sync(1);
      continue;
    }
    tc_fence_after();
    const int i = obs_row(a, u, s);
    const float c = c_smem[i < a.r ? i : 0];
    const int last = a.n - a.r + i;                     // last visible key of this row
    const int j0 = blk * kKeyTile;
    const bool full = j0 + kKeyTile - 1 <= a.n - a.r;   // every key of the tile is visible to every row
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * 128);
    float M = -INFINITY, Z = 0.f;
#pragma unroll 1
    for (int ch = 0; ch < 4; ++ch) {
      float v[32];
      tmem_ld32(taddr + ch * 32, v);
      if (!full) {
#pragma unroll
        for (int t = 0; t < 32; ++t)
          if (j0 + ch * 32 + t > last) v[t] = -INFINITY;
      }
      float mx = v[0];
#pragma unroll
      for (int t = 1; t < 32; ++t) mx = fmaxf(mx, v[t]);
      if (mx > -INFINITY) {
        const float m2 = mx * c;
        float z = 0.f;
#pragma unroll
        for (int t = 0; t < 32; ++t) z += fast_exp2(fmaf(v[t], c, -m2));
        if (m2 > M) {
          Z = Z * fast_exp2(M - m2) + z;
          M = m2;
        } else {
          Z += z * fast_exp2(m2 - M);
        }
      }
    }
    tc_fence_before();
    mbar_arrive(&bars->acc_empty[0][acc]);
    a.partial[((size_t)unit * a.n_blk + blk) * 128 + s] = make_float2(M, Z);
    __threadfence();
    group_sync(1);
    if (s == 0) bcast[0] = atomicAdd(&a.cnt[unit], 1);   // (a dead thread 0 has written -1 instead)
    group_sync(1);
    const bool last_partial = bcast[0] == a.n_blk - 1;
    group_sync(1);                                       // bcast may be rewritten after this point
    if (last_partial) {
      // this CTA delivered the row block's last tile: merge all partials of row s
      __threadfence();
      const float2* p = a.partial + (size_t)unit * a.n_blk * 128 + s;
      float Mx = -INFINITY;
      for (int t = 0; t < a.n_blk; ++t) Mx = fmaxf(Mx, __ldcg(&p[(size_t)t * 128]).x);
      float Zs = 0.f;
      for (int t = 0; t < a.n_blk; ++t) {
        const float2 e = __ldcg(&p[(size_t)t * 128]);
        if (e.y > 0.f) Zs += e.y * fast_exp2(e.x - Mx);
      }
      // 2^{c w - off} = softmax weight / G
      a.final_off[(size_t)unit * 128 + s] = Mx + log2f(Zs) + a.log2G;
      __threadfence();
      atomicAdd(&a.flag[unit], 1);       // the block is ready when all 128 rows have reported
    }
  }
}

// Pass-2 softmax group: thread `jl` owns key j0 + jl.
__device__ void column_sum_group(const TcArgs& a, Barriers* bars, uint32_t tmem_base, const float* c_smem,
                                 float2* row_const) {
  const int jl = threadIdx.x & 127, quarter = (threadIdx.x >> 5) & 3;
  int it = 0, prev_unit = -1;
  bool dead = false;     // a flag wait ran out: keep the pipeline protocol, skip the arithmetic
  bool gone = false;     // an accumulator wait ran out: keep only the group barriers
  UnitInfo u = unit_info(a, 0);
  for (TileWalk w(a); w.valid(); w.next(), ++it) {
    const int unit = w.t / a.n_blk, blk = w.t % a.n_blk;
    if (unit != prev_unit) {
      prev_unit = unit;
      u = unit_info(a, unit);
      if (!dead) {
        const long long t0 = now_ns();
        while (ld_acquire(&a.flag[unit]) < 128) {
          __nanosleep(200);
          if (now_ns() - t0 > kWaitLimitNs) {
            atomicExch(a.status, (int)AHAKV_ERR_TIMEOUT);
            dead = true;
            break;
          }
        }
      }
      group_sync(2);                                    // everyone is done with the previous constants
      if (jl < u.npad) {
        const int i = obs_row(a, u, jl);
        const bool live = jl < u.rows && !dead;
        row_const[jl] = make_float2(live ? c_smem[i] : 0.f,
                                    live ? __ldcg(&a.final_off[(size_t)unit * 128 + jl]) : INFINITY);
      }
      group_sync(2);
    }
    const int acc = it & 1, aph = (it >> 1) & 1;
    if (!gone && !mbar_wait(&bars->acc_full[1][acc], aph, a.status)) gone = true;
    if (gone) continue;  // only the unit-change barriers above remain
    tc_fence_after();
    const int j = blk * kKeyTile + jl;
    const bool full = blk * kKeyTile + kKeyTile - 1 <= a.n - a.r;
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((2 + acc) * 128);
    float sum = 0.f;
    // npad is a multiple of 16 and the product wrote exactly npad columns: never read beyond them.
    // Rows between `rows` and npad are zero rows of Q with weight 0 and offset +inf: 2^{-inf} = 0.
#pragma unroll 1
    for (int ch = 0; ch * 16 < u.npad; ++ch) {
      float v[16];
      tmem_ld16(taddr + ch * 16, v);
      if (full) {
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          const float2 rc = row_const[ch * 16 + t];
          sum += fast_exp2(fmaf(v[t], rc.x, -rc.y));
        }
      } else {
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          const int sr = ch * 16 + t;
          const float2 rc = row_const[sr];
          const bool vis = sr < u.rows && j <= a.n - a.r + obs_row(a, u, sr);
          if (vis) sum += fast_exp2(fmaf(v[t], rc.x, -rc.y));
        }
      }
    }
    tc_fence_before();
    mbar_arrive(&bars->acc_empty[1][acc]);
    if (j < a.n) a.s_raw[(size_t)unit * a.n + j] = sum;
  }
}

__global__ void __launch_bounds__(kThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap,
                const __grid_constant__ TcArgs a) {
  extern __shared__ char smem_raw[];
  char* tiles = reinterpret_cast<char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  char* q_smem[2] = {tiles, tiles + kQBytes + kKRingBytes};
  char* k_ring[2] = {tiles + kQBytes, tiles + 2 * kQBytes + kKRingBytes};
  char* misc = tiles + kSmemTiles;
  Barriers* bars = reinterpret_cast<Barriers*>(misc);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 256);
  int* bcast = reinterpret_cast<int*>(misc + 272);
  float* c_smem = reinterpret_cast<float*>(misc + 512);             // [256]
  float2* row_const = reinterpret_cast<float2*>(misc + 512 + 1024); // [128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = threadIdx.x; t < kMaxRows; t += kThreads) c_smem[t] = a.c[t];
  // Q rows a TMA box never covers (row blocks with fewer than 128 rows) must read as zeros, not as
  // whatever the last kernel left: zero both Q buffers once, before any bulk copy is issued.
  for (int p = 0; p < 2; ++p) {
    uint4* z = reinterpret_cast<uint4*>(q_smem[p]);
    for (int t = threadIdx.x; t < kQBytes / 16; t += kThreads) z[t] = make_uint4(0, 0, 0, 0);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (threadIdx.x == 0) {
    for (int p = 0; p < 2; ++p) {
      mbar_init(&bars->q_full[p], 1);
      for (int s = 0; s < kStages; ++s) {
        mbar_init(&bars->k_full[p][s], 1);
        mbar_init(&bars->k_empty[p][s], 1);
      }
      for (int s = 0; s < 2; ++s) {
        mbar_init(&bars->acc_full[p][s], 1);
        mbar_init(&bars->acc_empty[p][s], 128);
      }
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // all 512 TMEM columns: four 128-column accumulators
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(tmem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) producer(a, &qmap, &kmap, bars, 0, q_smem[0], k_ring[0]);
  } else if (warp == 1) {
    if (lane == 0) mma_issuer(a, bars, 0, q_smem[0], k_ring[0], tmem_base);
  } else if (warp == 2) {
    if (lane == 0) producer(a, &qmap, &kmap, bars, 1, q_smem[1], k_ring[1]);
  } else if (warp == 3) {
    if (lane == 0) mma_issuer(a, bars, 1, q_smem[1], k_ring[1], tmem_base);
  } else if (warp < 8) {
    row_stats_group(a, bars, tmem_base, c_smem, bcast);
  } else {
    column_sum_group(a, bars, tmem_base, c_smem, row_const);
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
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// 4-D map {d, tokens, heads, batch} with a {64, box_rows, box_heads, 1} box, 128-byte swizzle, zero fill.
bool make_map(CUtensorMap* m, const void* base, int bf16, int d, long long tokens, long long heads, long long batch,
              const long long stride[3], int es, int box_rows, int box_heads) {
  const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)batch};
  const cuuint64_t strides[3] = {(cuuint64_t)stride[2] * es, (cuuint64_t)stride[1] * es, (cuuint64_t)stride[0] * es};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_heads, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return encode_fn()(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
                     const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool score_tc_available() { return encode_fn() != nullptr; }

ahakv_status launch_score_tc(const Plan& pl, const void* q, const void* k, float* s_raw, float2* partial,
                             float* final_off, int* sync_words, int* status, cudaStream_t st) {
  static int n_sm = 0;
  static bool configured = false;
  if (!configured) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaFuncSetAttribute(score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
      return AHAKV_ERR_CUDA;
    configured = true;
  }
  const int units = pl.B * pl.Hkv * pl.n_rb;
  TcArgs a;
  a.n = pl.n; a.r = pl.r; a.G = pl.G; a.Hkv = pl.Hkv; a.n_rb = pl.n_rb; a.hb = pl.heads_per_rb;
  a.n_blk = pl.n_blk; a.D = pl.d;
  a.T = units * pl.n_blk;
  int ch = a.T / (n_sm * 8);
  a.CH = ch < 1 ? 1 : (ch > 4 ? 4 : ch);
  a.n_runs = (a.T + a.CH - 1) / a.CH;
  a.bf16 = pl.dtype == AHAKV_BF16;
  a.log2G = log2f((float)pl.G);
  for (int i = 0; i < kMaxRows; ++i) a.c[i] = pl.rows.c[i];
  a.partial = partial; a.final_off = final_off; a.s_raw = s_raw;
  a.cnt = sync_words; a.flag = sync_words + units; a.status = status;

  CUtensorMap qmap, kmap;
  const int q_box_rows = pl.r <= 128 ? pl.r : 128, q_box_heads = pl.r <= 128 ? pl.heads_per_rb : 1;
  if (!make_map(&qmap, q, a.bf16, pl.d, pl.r, pl.Hq, pl.B, pl.qs, pl.es, q_box_rows, q_box_heads) ||
      !make_map(&kmap, k, a.bf16, pl.d, pl.n, pl.Hkv, pl.B, pl.ks, pl.es, kKeyTile, 1))
    return AHAKV_ERR_CUDA;

  const int grid = a.n_runs < n_sm ? a.n_runs : n_sm;
  void* args[] = {&qmap, &kmap, &a};
  const cudaError_t e = cudaLaunchCooperativeKernel((const void*)score_tc_kernel, dim3(grid), dim3(kThreads), args,
                                                    (size_t)kSmemBytes, st);
  count_launch();
  if (e != cudaSuccess) return AHAKV_ERR_CUDA;
  return cuda_ok(cudaGetLastError());
}

}  // namespace ahakv
