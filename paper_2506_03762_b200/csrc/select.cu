// Value-prior refinement (Eq. 13-15) and budgeted selection (Algorithm 1).
//
// refine: one CTA per (sequence, KV head) adds the row-block partial scores,
//   smooths nu with the mean filter, normalises by the head-wide maximum,
//   multiplies, and adds the carried score.
// select: one CTA per (sequence, KV head) finds the B_s-th largest candidate
//   score with a 4 x 8-bit radix select on the order-preserving integer image of
//   the float, then emits, in ascending index order, every candidate above the
//   threshold plus the lowest-indexed ones equal to it, then the recent window.
#include "ahakv_internal.cuh"
#include "select_common.cuh"

namespace ahakv {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ float block_max(float x, float* red) {
#pragma unroll
  for (int o = 16; o; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = x;
  __syncthreads();
  float m = red[0];
  for (int w = 1; w < kWarps; ++w) m = fmaxf(m, red[w]);
  __syncthreads();
  return m;
}

__global__ void __launch_bounds__(kThreads) refine_kernel(const float* __restrict__ s_raw, const float* __restrict__ nu,
                                                          const float* __restrict__ prev, float* __restrict__ score,
                                                          const Shape pl, const int slots) {
  __shared__ float red[kWarps];
  const int unit = blockIdx.x, n = pl.n, half = pl.pool / 2;
  const bool prior = nu != nullptr;
  const float inv_w = 1.f / (float)pl.pool;
  const bool zero_pad = (pl.flags & AHAKV_FLAG_POOL_ZERO_PAD) != 0;
  const float* nu_u = prior ? nu + (size_t)unit * n : nullptr;
  float inv_gmax = 1.f;
  if (prior) {
    float m = 0.f;
    for (int j = threadIdx.x; j < n; j += kThreads) m = fmaxf(m, pooled(nu_u, j, n, half, inv_w, zero_pad));
    inv_gmax = __frcp_rn(block_max(m, red));
  }
  for (int j = threadIdx.x; j < n; j += kThreads) {
    float s = combine_slots(s_raw, (size_t)unit * slots * n + j, n, slots, pl.group_max);
    if (prior) s = __fmul_rn(__fmul_rn(pooled(nu_u, j, n, half, inv_w, zero_pad), inv_gmax), s);
    if (prev) s = __fadd_rn(s, prev[(size_t)unit * n + j]);
    score[(size_t)unit * n + j] = s;
  }
}

// The digit at which the count of keys, taken from the largest digit down, reaches `need`: a suffix scan of
// the 256-bin histogram by 256 threads.  Writes the extended prefix and how many keys of that digit are still
// needed; ends with a barrier.
template <int kCopies>
__device__ __forceinline__ void find_digit(const unsigned (*hist)[256], unsigned need, unsigned prefix, int shift,
                                           unsigned* out_prefix, unsigned* out_need, unsigned* warp_tot) {
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  unsigned h = 0, inc = 0;
  if (t < 256) {
#pragma unroll
    for (int c = 0; c < kCopies; ++c) h += hist[c][255 - t];   // thread t looks at digit 255 - t
    inc = h;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned x = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += x;
    }
    if (lane == 31) warp_tot[warp] = inc;
  }
  __syncthreads();
  if (t < 256) {
    for (int w = 0; w < warp; ++w) inc += warp_tot[w];
    if (inc >= need && inc - h < need) {       // exactly one digit crosses
      *out_prefix = prefix | ((unsigned)(255 - t) << shift);
      *out_need = need - (inc - h);
    }
  }
  __syncthreads();
}

// The budget of one (sequence, KV head): the call's, or the caller's own for this head, held to [max(Br, 1), Bud].
__device__ __forceinline__ int head_budget(const Shape& pl, const int32_t* budgets, int unit) {
  if (budgets == nullptr) return pl.Bud;
  return min(max(budgets[unit], max(pl.Br, 1)), pl.Bud);
}
// Entries of a head's index row beyond the tokens it keeps (heads with a budget of their own only).
__device__ __forceinline__ void pad_kept(int32_t* out, int kept_here, int n_keep) {
  for (int t = kept_here + threadIdx.x; t < n_keep; t += kThreads) out[t] = -1;
}

__global__ void __launch_bounds__(kThreads) select_kernel(const float* __restrict__ score, int32_t* __restrict__ kept,
                                                          const Shape pl, const int32_t* __restrict__ budgets) {
  __shared__ unsigned hist[1][256];
  __shared__ unsigned sh_prefix, sh_need, scan_tot[8];
  __shared__ int warp_gt[kWarps], warp_eq[kWarps];
  __shared__ int run_gt, run_eq;
  const int unit = blockIdx.x, n = pl.n;
  const float* s = score + (size_t)unit * n;
  int32_t* out = kept + (size_t)unit * pl.n_keep;
  const int bud = head_budget(pl, budgets, unit);
  pad_kept(out, min(n, bud), pl.n_keep);
  if (n <= bud) {                          // nothing to evict
    for (int j = threadIdx.x; j < n; j += kThreads) out[j] = j;
    return;
  }
  const int n_cand = n - pl.Br, Bs = bud - pl.Br;
  for (int t = threadIdx.x; t < pl.Br; t += kThreads) out[Bs + t] = n_cand + t;   // recent window
  if (Bs == 0) return;

  // ---- radix select: key of the Bs-th largest candidate --------------------
  unsigned prefix = 0, need = (unsigned)Bs;     // `need` elements still to take among keys matching prefix
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const unsigned mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    if (threadIdx.x < 256) hist[0][threadIdx.x] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < n_cand; j += kThreads) {
      const unsigned key = order_key(s[j]);
      if ((key & mask) == prefix) atomicAdd(&hist[0][(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    find_digit<1>(hist, need, prefix, shift, &sh_prefix, &sh_need, scan_tot);
    prefix = sh_prefix;
    need = sh_need;
    __syncthreads();
  }
  const unsigned thr = prefix;              // exact key of the threshold score
  const int need_eq = (int)need;            // how many keys equal to thr are kept (lowest index first)

  // ---- ordered emission ------------------------------------------------------
  if (threadIdx.x == 0) { run_gt = 0; run_eq = 0; }
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < n_cand; base += kThreads) {
    const int j = base + threadIdx.x;
    bool gt = false, eq = false;
    if (j < n_cand) {
      const unsigned key = order_key(s[j]);
      gt = key > thr;
      eq = key == thr;
    }
    const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    const unsigned below = (1u << lane) - 1u;
    if (lane == 0) { warp_gt[warp] = __popc(bg); warp_eq[warp] = __popc(be); }
    __syncthreads();
    int gt_before = run_gt + __popc(bg & below), eq_before = run_eq + __popc(be & below);
    for (int w = 0; w < warp; ++w) { gt_before += warp_gt[w]; eq_before += warp_eq[w]; }
    if (gt || (eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = j;
    __syncthreads();
    if (threadIdx.x == kThreads - 1) {
      run_gt = gt_before + (gt ? 1 : 0);
      run_eq = eq_before + (eq ? 1 : 0);
    }
    __syncthreads();
  }
}

// Refinement and selection of one (sequence, KV head) in one CTA, for n <= kPer * kThreads.  Thread t owns
// tokens t, t + kThreads, t + 2 kThreads, ... (coalesced) and keeps their refined scores in registers from the
// first load to the last store: the value prior is applied once, and the four radix passes and the ordered
// emission never go back to memory.  Same arithmetic, in the same order, as refine_kernel and select_kernel.
// kPer is the number of tokens a thread owns (every loop below is unrolled over it, so a short context is not
// made to pay for the longest one).
constexpr int kPerMax = 32;
constexpr int kHistCopies = 4;

template <int kPer, bool kPrev>
__global__ void __launch_bounds__(kThreads, 1) refine_select_kernel(const float* __restrict__ s_raw,
                                                                    const float* __restrict__ nu,
                                                                    const float* __restrict__ prev,
                                                                    float* __restrict__ score, int32_t* __restrict__ kept,
                                                                    const Shape pl, const int slots,
                                                                    const int32_t* __restrict__ budgets) {
  __shared__ float red[kWarps];
  // four copies of the histogram, one per quarter of the warps: in the first passes nearly all keys of a head fall
  // into one or two bins, and the atomics on one counter are served one after the other
  __shared__ unsigned hist[kHistCopies][256];
  __shared__ unsigned sh_prefix, sh_need, scan_tot[8];
  __shared__ int2 cnt[kPer * kWarps];      // kept-candidate counts (greater, equal) per 32-token group, in token order
  const int unit = blockIdx.x, n = pl.n, half = pl.pool / 2;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool prior = nu != nullptr;
  const float inv_w = 1.f / (float)pl.pool;
  const bool zero_pad = (pl.flags & AHAKV_FLAG_POOL_ZERO_PAD) != 0;
  const float* nu_u = prior ? nu + (size_t)unit * n : nullptr;

  uint32_t key[kPer];                                       // first the bits of gamma, then the score's order key
  float inv_gmax = 1.f;
  if (prior) {
    // the head's value norms go to shared memory in one coalesced sweep; the mean filter reads them there
    extern __shared__ float nu_s[];
    {
      float v[kPer];
#pragma unroll
      for (int e = 0; e < kPer; ++e) {
        const int j = e * kThreads + threadIdx.x;
        v[e] = j < n ? nu_u[j] : 0.f;
      }
#pragma unroll
      for (int e = 0; e < kPer; ++e) {
        const int j = e * kThreads + threadIdx.x;
        if (j < n) nu_s[j] = v[e];
      }
    }
    __syncthreads();
    float m = 0.f;
#pragma unroll
    for (int e = 0; e < kPer; ++e) {
      const int j = e * kThreads + threadIdx.x;
      const float g = j < n ? pooled(nu_s, j, n, half, inv_w, zero_pad) : 0.f;
      key[e] = __float_as_uint(g);
      m = fmaxf(m, g);
    }
    inv_gmax = __frcp_rn(block_max(m, red));
  }
  // loads in flight at a time: without a carried score, and with fewer than 32 keys to hold, the registers allow
  // twice as many
  constexpr int kWide = (kPrev || kPer > 16) ? 8 : 16;
  constexpr int kBatch = kPer < kWide ? kPer : kWide;
#pragma unroll
  for (int e0 = 0; e0 < kPer; e0 += kBatch) {              // eight tokens' loads in flight at a time
    float sr[kBatch], pv[kBatch];
#pragma unroll
    for (int e = 0; e < kBatch; ++e) {
      const int j = (e0 + e) * kThreads + threadIdx.x;
      sr[e] = 0.f; pv[e] = 0.f;
      if (j < n) {
        sr[e] = combine_slots(s_raw, (size_t)unit * slots * n + j, n, slots, pl.group_max);
        if (kPrev) pv[e] = prev[(size_t)unit * n + j];
      }
    }
#pragma unroll
    for (int e = 0; e < kBatch; ++e) {
      const int j = (e0 + e) * kThreads + threadIdx.x;
      const float g = prior ? __uint_as_float(key[e0 + e]) : 0.f;
      key[e0 + e] = 0u;
      if (j < n) {
        float s = sr[e];
        if (prior) s = __fmul_rn(__fmul_rn(g, inv_gmax), s);
        if (kPrev) s = __fadd_rn(s, pv[e]);
        score[(size_t)unit * n + j] = s;
        key[e0 + e] = order_key(s);
      }
    }
  }

  int32_t* out = kept + (size_t)unit * pl.n_keep;
  const int bud = head_budget(pl, budgets, unit);
  pad_kept(out, min(n, bud), pl.n_keep);
  if (n <= bud) {                          // nothing to evict
#pragma unroll
    for (int e = 0; e < kPer; ++e)
      if (e * kThreads + threadIdx.x < n) out[e * kThreads + threadIdx.x] = e * kThreads + threadIdx.x;
    return;
  }
  const int n_cand = n - pl.Br, Bs = bud - pl.Br;
  for (int t = threadIdx.x; t < pl.Br; t += kThreads) out[Bs + t] = n_cand + t;   // recent window
  if (Bs == 0) return;

  // ---- radix select on the keys in registers: key of the Bs-th largest candidate ----
  unsigned prefix = 0, need = (unsigned)Bs;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const unsigned mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    static_assert(kHistCopies * 256 == kThreads, "one counter per thread to clear");
    hist[threadIdx.x >> 8][threadIdx.x & 255] = 0;
    __syncthreads();
#pragma unroll
    for (int e = 0; e < kPer; ++e) {
      const bool in = e * kThreads + (int)threadIdx.x < n_cand && (key[e] & mask) == prefix;
      const unsigned digit = (key[e] >> shift) & 255u;
      unsigned* bins = hist[warp & (kHistCopies - 1)];
      if (pass == 0) {
        // sign and high exponent bits: nearly all scores of a head share one digit, and atomics on one counter
        // are served one after the other.  One atomic for the warp when all its digits agree.
        const unsigned live = __ballot_sync(0xffffffffu, in);
        const unsigned first = __shfl_sync(0xffffffffu, digit, live ? __ffs(live) - 1 : 0);
        if (__all_sync(0xffffffffu, !in || digit == first)) {
          if (live && lane == __ffs(live) - 1) atomicAdd(&bins[digit], (unsigned)__popc(live));
        } else if (in) {
          atomicAdd(&bins[digit], 1u);
        }
      } else if (in) {                         // later digits are spread out, and ever fewer tokens are still in
        atomicAdd(&bins[digit], 1u);
      }
    }
    __syncthreads();
    find_digit<kHistCopies>(hist, need, prefix, shift, &sh_prefix, &sh_need, scan_tot);
    prefix = sh_prefix;
    need = sh_need;
    __syncthreads();
  }
  const unsigned thr = prefix;
  const int need_eq = (int)need;

  // ---- ordered emission: counts per 32-token group, one scan over the groups, then the writes ----
#pragma unroll
  for (int e = 0; e < kPer; ++e) {
    const bool c = e * kThreads + (int)threadIdx.x < n_cand;
    const unsigned bg = __ballot_sync(0xffffffffu, c && key[e] > thr), be = __ballot_sync(0xffffffffu, c && key[e] == thr);
    if (lane == 0) cnt[e * kWarps + warp] = make_int2(__popc(bg), __popc(be));
  }
  __syncthreads();
  {
    // exclusive scan of the kPer * kWarps (<= kThreads) group counts, in place: thread t owns group t
    const bool mine = (int)threadIdx.x < kPer * kWarps;
    const int2 v = mine ? cnt[threadIdx.x] : make_int2(0, 0);
    int2 inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, inc.x, o), y = __shfl_up_sync(0xffffffffu, inc.y, o);
      if (lane >= o) { inc.x += x; inc.y += y; }
    }
    __shared__ int2 warp_tot[kWarps];
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    int2 base = make_int2(0, 0);
    for (int w = 0; w < warp; ++w) { base.x += warp_tot[w].x; base.y += warp_tot[w].y; }
    if (mine) cnt[threadIdx.x] = make_int2(base.x + inc.x - v.x, base.y + inc.y - v.y);
    __syncthreads();
  }
  const unsigned below = (1u << lane) - 1u;
#pragma unroll
  for (int e = 0; e < kPer; ++e) {
    const int j = e * kThreads + threadIdx.x;
    const bool c = j < n_cand;
    const bool gt = c && key[e] > thr, eq = c && key[e] == thr;
    const unsigned bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
    const int2 b0 = cnt[e * kWarps + warp];
    const int gt_before = b0.x + __popc(bg & below), eq_before = b0.y + __popc(be & below);
    if (gt || (eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = j;
  }
}

}  // namespace

ahakv_status launch_refine(const Plan& pl, const float* s_raw, const float* nu, const float* score_prev,
                           float* score, int slots, cudaStream_t st) {
  refine_kernel<<<pl.B * pl.Hkv, kThreads, 0, st>>>(s_raw, nu, score_prev, score, pl, slots);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

ahakv_status launch_select(const Plan& pl, const float* score, int32_t* kept_idx, const int32_t* budgets,
                           cudaStream_t st) {
  select_kernel<<<pl.B * pl.Hkv, kThreads, 0, st>>>(score, kept_idx, pl, budgets);
  count_launch();
  return cuda_ok(cudaGetLastError());
}


// Both steps in one launch when a head's scores fit in the registers of one CTA; false if they do not.
bool refine_select_fits(const Plan& pl) { return pl.n <= kPerMax * kThreads; }

namespace {
template <int kPer, bool kPrev>
ahakv_status launch_refine_select_as(const Plan& pl, const float* s_raw, const float* nu, const float* score_prev,
                                     float* score, int32_t* kept_idx, int slots, const int32_t* budgets,
                                     cudaStream_t st) {
  // Static and dynamic shared memory together may pass 48 KB well before the dynamic part alone does, and
  // beyond that the launch needs leave, asked for once per device: ask whenever the value norms are staged.
  constexpr int kMaxDevices = 64;
  static bool configured[kMaxDevices] = {};
  const size_t smem = nu ? (size_t)pl.n * sizeof(float) : 0;
  if (smem > 0) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AHAKV_ERR_CUDA;
    if (!configured[dev]) {
      if (cudaFuncSetAttribute(refine_select_kernel<kPer, kPrev>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               kPer * kThreads * (int)sizeof(float)) != cudaSuccess)
        return AHAKV_ERR_CUDA;
      configured[dev] = true;
    }
  }
  refine_select_kernel<kPer, kPrev><<<pl.B * pl.Hkv, kThreads, smem, st>>>(s_raw, nu, score_prev, score, kept_idx, pl,
                                                                    slots, budgets);
  count_launch();
  return cuda_ok(cudaGetLastError());
}
}  // namespace

ahakv_status launch_refine_select(const Plan& pl, const float* s_raw, const float* nu, const float* score_prev,
                                  float* score, int32_t* kept_idx, int slots, const int32_t* budgets,
                                  cudaStream_t st) {
  const int per = (pl.n + kThreads - 1) / kThreads;          // tokens a thread owns
  if (score_prev) {
    if (per <= 4) return launch_refine_select_as<4, true>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
    if (per <= 8) return launch_refine_select_as<8, true>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
    if (per <= 16) return launch_refine_select_as<16, true>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
    return launch_refine_select_as<kPerMax, true>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
  }
  if (per <= 4) return launch_refine_select_as<4, false>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
  if (per <= 8) return launch_refine_select_as<8, false>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
  if (per <= 16) return launch_refine_select_as<16, false>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
  return launch_refine_select_as<kPerMax, false>(pl, s_raw, nu, score_prev, score, kept_idx, slots, budgets, st);
}

}  // namespace ahakv
