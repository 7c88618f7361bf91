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

__device__ __forceinline__ float pooled(const float* __restrict__ nu, int j, int n, int half, float inv_full) {
  const int lo = max(j - half, 0), hi = min(j + half, n - 1);
  float s = 0.f;
  for (int t = lo; t <= hi; ++t) s += nu[t];
  return inv_full > 0.f ? s * inv_full : s / (float)(hi - lo + 1);
}

__global__ void __launch_bounds__(kThreads) refine_kernel(const float* __restrict__ s_raw, const float* __restrict__ nu,
                                                          const float* __restrict__ prev, float* __restrict__ score,
                                                          const Plan pl, const int slots) {
  __shared__ float red[kWarps];
  const int unit = blockIdx.x, n = pl.n, half = pl.pool / 2;
  const bool prior = nu != nullptr;
  const float inv_full = (pl.flags & AHAKV_FLAG_POOL_ZERO_PAD) ? 1.f / (float)pl.pool : 0.f;
  const float* nu_u = prior ? nu + (size_t)unit * n : nullptr;
  float gmax = 1.f;
  if (prior) {
    float m = 0.f;
    for (int j = threadIdx.x; j < n; j += kThreads) m = fmaxf(m, pooled(nu_u, j, n, half, inv_full));
    gmax = block_max(m, red);
  }
  for (int j = threadIdx.x; j < n; j += kThreads) {
    float s = s_raw[(size_t)unit * slots * n + j];
    for (int t = 1; t < slots; ++t) s += s_raw[((size_t)unit * slots + t) * n + j];
    if (prior) s = (pooled(nu_u, j, n, half, inv_full) / gmax) * s;
    if (prev) s += prev[(size_t)unit * n + j];
    score[(size_t)unit * n + j] = s;
  }
}

// Monotone map float -> uint32: a > b  <=>  key(a) > key(b) (for non-NaN values).
__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(kThreads) select_kernel(const float* __restrict__ score, int32_t* __restrict__ kept,
                                                          const Plan pl) {
  __shared__ unsigned hist[256];
  __shared__ unsigned sh_prefix, sh_need;
  __shared__ int warp_gt[kWarps], warp_eq[kWarps];
  __shared__ int run_gt, run_eq;
  const int unit = blockIdx.x, n = pl.n;
  const float* s = score + (size_t)unit * n;
  int32_t* out = kept + (size_t)unit * pl.n_keep;
  if (n <= pl.Bud) {                       // nothing to evict
    for (int j = threadIdx.x; j < n; j += kThreads) out[j] = j;
    return;
  }
  const int n_cand = n - pl.Br, Bs = pl.Bs;
  for (int t = threadIdx.x; t < pl.Br; t += kThreads) out[Bs + t] = n_cand + t;   // recent window
  if (Bs == 0) return;

  // ---- radix select: key of the Bs-th largest candidate --------------------
  unsigned prefix = 0, need = (unsigned)Bs;     // `need` elements still to take among keys matching prefix
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const unsigned mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < n_cand; j += kThreads) {
      const unsigned key = order_key(s[j]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned acc = 0;
      int dgt = 255;
      for (; dgt > 0; --dgt) {
        if (acc + hist[dgt] >= need) break;
        acc += hist[dgt];
      }
      sh_prefix = prefix | ((unsigned)dgt << shift);
      sh_need = need - acc;                 // taken from the bucket `dgt`
    }
    __syncthreads();
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

}  // namespace

ahakv_status launch_refine(const Plan& pl, const float* s_raw, const float* nu, const float* score_prev,
                           float* score, cudaStream_t st) {
  refine_kernel<<<pl.B * pl.Hkv, kThreads, 0, st>>>(s_raw, nu, score_prev, score, pl, pl.use_tc ? pl.n_rb : 1);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

ahakv_status launch_select(const Plan& pl, const float* score, int32_t* kept_idx, cudaStream_t st) {
  select_kernel<<<pl.B * pl.Hkv, kThreads, 0, st>>>(score, kept_idx, pl);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace ahakv
