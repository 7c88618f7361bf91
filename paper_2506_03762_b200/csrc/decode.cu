// The generation phase one token at a time (Algorithm 1, Generation: A = q_t K^T, F_t = SGsoftmax(A) + F_{t-1},
// then S = TopK(F_t, B_s) U recent B_r and K <- K_S, V <- V_S before the next token).
//
// step_score_kernel: one CTA per (sequence, KV head).  The G query rows of the group (one new query per head)
//   against the n cached keys is a matrix-vector product, bound by reading K once.  16-bit inputs: warp-level
//   m16n8k16 products, the heads on the rows and eight keys on the columns (step_logits_mma).  float32 inputs:
//   half a warp (or a quarter, by row size) reads one key row with 16-byte loads, every lane keeps its slice of
//   the G queries in registers, and the partial dot products meet by shuffle.  The G x n logits stay in shared
//   memory; row maxima and sums are block reductions in a fixed order; the new score is written in one more sweep.
//   No scratch memory, no second read of K.
//
// step_slots_kernel: the same, for a cache kept as slots: it also copies the new token's rows into the free slot
//   and names the slot that becomes free (smallest score outside the recent window).
//
// compact_inplace_kernel: one CTA per (sequence, KV head).  kept_idx is ascending, so row t of the result comes
//   from row kept_idx[t] >= t: rows before the first evicted index do not move at all, and the others move in
//   batches through shared memory (all loads of a batch, a barrier, all its stores), so no row is overwritten
//   before it has been read.
#include <type_traits>

#include "ahakv_internal.cuh"
#include "mma_sync.cuh"
#include "select_common.cuh"

namespace ahakv {
namespace {

constexpr int kStepThreads = 512;
constexpr int kStepMaxG = 16;                  // query heads per KV head the step kernel takes
constexpr size_t kStepMaxLogitBytes = 160 * 1024;   // 40960 logits

template <typename T> using Acc = typename std::conditional<std::is_same<T, float>::value, double, float>::type;

// The G x n logits of one (sequence, KV head), in log2 units, into shared memory.  LANES threads share a key row
// (16 bytes each); kG query heads.
template <typename T, int D, int kG>
__device__ __forceinline__ void step_logits(const T* __restrict__ q, const T* __restrict__ k, const Shape& pl, int b,
                                            int h, Acc<T> c, float* logit) {
  using A = Acc<T>;
  constexpr int V = Vec16<T>::N, LANES = D / V, KEYS_PER_WARP = 32 / LANES;
  const int n = pl.n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, sub = lane % LANES, which = lane / LANES;

  // this lane's slice of each of the group's queries
  float qreg[kG][V];
#pragma unroll
  for (int g = 0; g < kG; ++g) {
    const T* row = q + (long long)b * pl.qs[0] + (long long)(h * pl.G + g) * pl.qs[1];
    Vec16<T>::widen(*reinterpret_cast<const uint4*>(row + sub * V), qreg[g]);
  }
  const T* kbase = k + (long long)b * pl.ks[0] + (long long)h * pl.ks[1];
  constexpr int kUnroll = 4;                                     // key rows in flight per lane
  const int stride = (kStepThreads / 32) * KEYS_PER_WARP;
  for (int j0 = warp * KEYS_PER_WARP + which; j0 - which < n; j0 += stride * kUnroll) {
    uint4 raw[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = j0 + u * stride;
      raw[u] = j < n ? *reinterpret_cast<const uint4*>(kbase + (long long)j * pl.ks[2] + sub * V) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = j0 + u * stride;
      float kv[V];
      Vec16<T>::widen(raw[u], kv);
#pragma unroll
      for (int g = 0; g < kG; ++g) {
        A acc = 0;
#pragma unroll
        for (int e = 0; e < V; ++e) acc = fma((A)qreg[g][e], (A)kv[e], acc);
#pragma unroll
        for (int o = LANES / 2; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (sub == 0 && j < n) logit[g * n + j] = (float)(acc * c);    // log2 units
      }
    }
  }
  __syncthreads();
}

// The same logits for 16-bit inputs on the warp-level tensor-core instruction: a G x n by d product is far too
// thin for the tensor memory path, but the FP32 multiply-add loop above spends forty-odd instructions a key on
// conversions and shuffle reductions, and mma.sync m16n8k16 (heads on the 16 rows, 8 keys on the columns, FP32
// accumulation of exact products) spends three.  The sum over d does not care in which order d is walked, so each
// thread takes one contiguous quarter of a row -- of its query head's row for the A operand, of its key's row for the
// B operand -- and hands its 32-bit words to the instruction in pairs: the k-slices the four threads of a group
// present side by side are then the same permutation of d for A and for B.
template <typename T, int D, int kG>
__device__ __forceinline__ void step_logits_mma(const T* __restrict__ q, const T* __restrict__ k, const Shape& pl, int b,
                                                int h, float c, float* logit) {
  constexpr int CH = D / 4, W = CH / 2, Q4 = CH / 8;           // a thread's quarter row: elements, 32-bit words, 16-byte loads
  constexpr int kSteps = D / 16, kUnroll = 4, kWarps = kStepThreads / 32;
  const int n = pl.n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, grp = lane >> 2, tig = lane & 3;

  // A: head `grp` (and `grp + 8` when there are more than eight) of the group's queries, this thread's quarter
  uint32_t qa[W], qb[W];
#pragma unroll
  for (int t = 0; t < W; ++t) { qa[t] = 0u; qb[t] = 0u; }
  if (grp < kG) {
    const T* row = q + (long long)b * pl.qs[0] + (long long)(h * pl.G + grp) * pl.qs[1] + CH * tig;
#pragma unroll
    for (int t = 0; t < Q4; ++t) {
      const uint4 u = *reinterpret_cast<const uint4*>(row + 8 * t);
      qa[4 * t] = u.x; qa[4 * t + 1] = u.y; qa[4 * t + 2] = u.z; qa[4 * t + 3] = u.w;
    }
  }
  if (kG > 8 && grp + 8 < kG) {
    const T* row = q + (long long)b * pl.qs[0] + (long long)(h * pl.G + grp + 8) * pl.qs[1] + CH * tig;
#pragma unroll
    for (int t = 0; t < Q4; ++t) {
      const uint4 u = *reinterpret_cast<const uint4*>(row + 8 * t);
      qb[4 * t] = u.x; qb[4 * t + 1] = u.y; qb[4 * t + 2] = u.z; qb[4 * t + 3] = u.w;
    }
  }
  const T* kbase = k + (long long)b * pl.ks[0] + (long long)h * pl.ks[1] + CH * tig;
  const int n_blocks = (n + 7) / 8;
  for (int blk0 = warp; blk0 < n_blocks; blk0 += kWarps * kUnroll) {
    uint4 raw[kUnroll][Q4];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j = (blk0 + u * kWarps) * 8 + grp;               // this thread's key in block u
#pragma unroll
      for (int t = 0; t < Q4; ++t)
        raw[u][t] = j < n ? *reinterpret_cast<const uint4*>(kbase + (long long)j * pl.ks[2] + 8 * t) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int j0 = (blk0 + u * kWarps) * 8;
      if (j0 >= n) break;                                        // uniform over the warp
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int t = 0; t < Q4; ++t) {
        const uint32_t w[4] = {raw[u][t].x, raw[u][t].y, raw[u][t].z, raw[u][t].w};
        // two k-steps a 16-byte load: words (0, 1) and (2, 3)
        Mma16816<T>::run(acc, qa[4 * t], qb[4 * t], qa[4 * t + 1], qb[4 * t + 1], w[0], w[1]);
        Mma16816<T>::run(acc, qa[4 * t + 2], qb[4 * t + 2], qa[4 * t + 3], qb[4 * t + 3], w[2], w[3]);
      }
      static_assert(kSteps == 2 * Q4, "two k-steps per 16-byte load");
      const int j = j0 + 2 * tig;
      if (grp < kG) {
        if (j < n) logit[grp * n + j] = acc[0] * c;
        if (j + 1 < n) logit[grp * n + j + 1] = acc[1] * c;
      }
      if (kG > 8 && grp + 8 < kG) {
        if (j < n) logit[(grp + 8) * n + j] = acc[2] * c;
        if (j + 1 < n) logit[(grp + 8) * n + j + 1] = acc[3] * c;
      }
    }
  }
  __syncthreads();
}

template <typename T, int D, int kG>
__device__ __forceinline__ void step_logits_any(const T* __restrict__ q, const T* __restrict__ k, const Shape& pl, int b,
                                                int h, double c_row, float* logit) {
  if constexpr (std::is_same<T, float>::value) step_logits<T, D, kG>(q, k, pl, b, h, (Acc<T>)c_row, logit);
  else step_logits_mma<T, D, kG>(q, k, pl, b, h, (float)c_row, logit);
}

// kG block-wide reductions at once, each in a fixed order: warp shuffles, then the warps' results in warp order.
template <bool kMax, int kG>
__device__ __forceinline__ void block_reduce_heads(float (&x)[kG], float (*red)[kStepThreads / 32]) {
#pragma unroll
  for (int g = 0; g < kG; ++g) {
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      const float y = __shfl_xor_sync(0xffffffffu, x[g], o);
      x[g] = kMax ? fmaxf(x[g], y) : x[g] + y;
    }
  }
  __syncthreads();                              // `red` may still be read from the last reduction
  if ((threadIdx.x & 31) == 0) {
#pragma unroll
    for (int g = 0; g < kG; ++g) red[g][threadIdx.x >> 5] = x[g];
  }
  __syncthreads();
#pragma unroll
  for (int g = 0; g < kG; ++g) {
    float r = red[g][0];
    for (int w = 1; w < kStepThreads / 32; ++w) r = kMax ? fmaxf(r, red[g][w]) : r + red[g][w];
    x[g] = r;
  }
}

// All query heads at once: shift and normaliser of every head, 2^{x - M} in place of the logits, and the factor
// 1 / (G Z) of each head in w[].
template <int kG>
__device__ __forceinline__ void step_weights(float* logit, int n, float inv_g, float (*red)[kStepThreads / 32],
                                             float (&w)[kG]) {
  float m[kG];
#pragma unroll
  for (int g = 0; g < kG; ++g) m[g] = -INFINITY;
  for (int j = threadIdx.x; j < n; j += kStepThreads) {
#pragma unroll
    for (int g = 0; g < kG; ++g) m[g] = fmaxf(m[g], logit[g * n + j]);
  }
  block_reduce_heads<true, kG>(m, red);
  float z[kG];
#pragma unroll
  for (int g = 0; g < kG; ++g) z[g] = 0.f;
  for (int j = threadIdx.x; j < n; j += kStepThreads) {
#pragma unroll
    for (int g = 0; g < kG; ++g) {
      const float e = fast_exp2(logit[g * n + j] - m[g]);
      logit[g * n + j] = e;                     // read back by the same thread only
      z[g] += e;
    }
  }
  block_reduce_heads<false, kG>(z, red);
#pragma unroll
  for (int g = 0; g < kG; ++g) w[g] = inv_g / z[g];
}

// Token j's share of the step: the weights of the group's heads pooled.
template <int kG>
__device__ __forceinline__ float step_pooled(const float* logit, int n, int j, int group_max, const float (&w)[kG]) {
  float s = logit[j] * w[0];
#pragma unroll
  for (int g = 1; g < kG; ++g) {
    const float t = logit[g * n + j] * w[g];
    s = group_max ? fmaxf(s, t) : s + t;
  }
  return s;
}

template <typename T, int D, int kG>
__global__ void __launch_bounds__(kStepThreads) step_score_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                                  const float* __restrict__ prev,
                                                                  float* __restrict__ score, const Shape pl,
                                                                  const double c_row) {
  extern __shared__ __align__(16) float logit[];                 // [kG][n]
  __shared__ float red[kG][kStepThreads / 32];
  const int unit = blockIdx.x, b = unit / pl.Hkv, h = unit % pl.Hkv, n = pl.n;
  step_logits_any<T, D, kG>(q, k, pl, b, h, c_row, logit);
  float w[kG];
  step_weights<kG>(logit, n, pl.group_max ? 1.f : 1.f / (float)kG, red, w);
  for (int j = threadIdx.x; j < n; j += kStepThreads) {
    float s = step_pooled<kG>(logit, n, j, pl.group_max, w);
    if (prev) s = __fadd_rn(s, prev[(size_t)unit * n + j]);
    score[(size_t)unit * n + j] = s;
  }
}

// One generation step on a cache kept as slots (no row ever moves): the new token's key and value rows go into the
// free slot of the (sequence, KV head), the one new query per head is scored against every slot, the score is
// updated in place, and the slot with the smallest score outside the recent window -- of equal scores the most recent
// token -- is declared free for the next step.  `pos` holds the logical position of the token in each slot; the
// recent window is the recent_window largest positions, the new token's included.
template <typename T, int D, int kG>
__global__ void __launch_bounds__(kStepThreads) step_slots_kernel(const T* __restrict__ q, const T* __restrict__ k_new,
                                                                  const T* __restrict__ v_new, T* __restrict__ k,
                                                                  T* __restrict__ v, float* __restrict__ score,
                                                                  int32_t* __restrict__ pos, int32_t* __restrict__ free_slot,
                                                                  const Shape pl, const double c_row, const int new_pos) {
  extern __shared__ __align__(16) float logit[];                 // [kG][n]
  __shared__ float red[kG][kStepThreads / 32];
  __shared__ unsigned long long best[kStepThreads / 32];
  constexpr int V = Vec16<T>::N, LANES = D / V;
  const int unit = blockIdx.x, b = unit / pl.Hkv, h = unit % pl.Hkv, n = pl.n;
  float* sc = score + (size_t)unit * n;
  int32_t* ps = pos + (size_t)unit * n;
  const int slot = free_slot[unit];
  if (slot < 0 || slot >= n) return;                             // the caller's table is broken: touch nothing
  // the new token moves in
  if (threadIdx.x < 2 * LANES) {
    const int sub = threadIdx.x % LANES;
    const bool is_v = threadIdx.x >= LANES;
    const T* src = (is_v ? v_new : k_new) + ((long long)b * pl.Hkv + h) * D + sub * V;
    T* dst = is_v ? v + (long long)b * pl.vs[0] + (long long)h * pl.vs[1] + (long long)slot * pl.vs[2] + sub * V
                  : k + (long long)b * pl.ks[0] + (long long)h * pl.ks[1] + (long long)slot * pl.ks[2] + sub * V;
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  }
  __syncthreads();                                               // the row is read back by other threads below
  step_logits_any<T, D, kG>(q, k, pl, b, h, c_row, logit);
  float w[kG];
  step_weights<kG>(logit, n, pl.group_max ? 1.f : 1.f / (float)kG, red, w);
  // F_t = SGsoftmax(A_t) + F_{t-1}, and the candidate to leave: smallest score, then largest position
  const int oldest_protected = new_pos - pl.Br + 1;             // positions from here on are the recent window
  unsigned long long mine = ~0ull;
  for (int j = threadIdx.x; j < n; j += kStepThreads) {
    float s = step_pooled<kG>(logit, n, j, pl.group_max, w);
    const int pj = j == slot ? new_pos : ps[j];
    if (j != slot) s = __fadd_rn(s, sc[j]);                      // a new token starts at zero
    sc[j] = s;
    if (pj < oldest_protected) {
      // ascending in (score, -position): the position is below 2^31, so ~pj orders it downwards within 32 bits
      const unsigned long long key = ((unsigned long long)order_key(s) << 32) | (unsigned)(0x7fffffff - pj);
      if (key < mine) mine = key;
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    const unsigned long long y = __shfl_xor_sync(0xffffffffu, mine, o);
    if (y < mine) mine = y;
  }
  if ((threadIdx.x & 31) == 0) best[threadIdx.x >> 5] = mine;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long m = best[0];
    for (int w = 1; w < kStepThreads / 32; ++w) if (best[w] < m) m = best[w];
    best[0] = m;
  }
  __syncthreads();
  const unsigned long long win = best[0];
  if (win == ~0ull) {                                            // no slot outside the recent window: a broken position table
    if (threadIdx.x == 0) free_slot[unit] = -1;
    return;
  }
  const int win_pos = 0x7fffffff - (int)(unsigned)(win & 0xffffffffu);
  for (int j = threadIdx.x; j < n; j += kStepThreads) {
    const int pj = j == slot ? new_pos : ps[j];
    if (j == slot) ps[j] = new_pos;
    if (pj == win_pos) {                                         // positions are distinct: exactly one slot
      ps[j] = -1;
      free_slot[unit] = j;
    }
  }
}

template <typename T, int D, int kG>
ahakv_status launch_step_as(const Plan& pl, const void* q, const void* k, const float* prev, float* score,
                            cudaStream_t st) {
  const size_t smem = (size_t)kG * pl.n * sizeof(float);
  constexpr int kMaxDevices = 64;
  static size_t configured[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AHAKV_ERR_CUDA;
  if (smem > 40 * 1024 && configured[dev] < kStepMaxLogitBytes) {
    if (cudaFuncSetAttribute(step_score_kernel<T, D, kG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kStepMaxLogitBytes) != cudaSuccess)
      return AHAKV_ERR_CUDA;
    configured[dev] = kStepMaxLogitBytes;
  }
  const Shape& shape = pl;
  step_score_kernel<T, D, kG><<<pl.B * pl.Hkv, kStepThreads, smem, st>>>((const T*)q, (const T*)k, prev, score, shape,
                                                                      pl.lambda[0] * 1.4426950408889634);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

template <typename T, int D, int kG>
ahakv_status launch_slots_as(const Plan& pl, const void* q, const void* k_new, const void* v_new, void* k, void* v,
                             float* score, int32_t* pos, int32_t* free_slot, int new_pos, cudaStream_t st) {
  const size_t smem = (size_t)kG * pl.n * sizeof(float);
  constexpr int kMaxDevices = 64;
  static size_t configured[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AHAKV_ERR_CUDA;
  if (smem > 40 * 1024 && configured[dev] < kStepMaxLogitBytes) {
    if (cudaFuncSetAttribute(step_slots_kernel<T, D, kG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kStepMaxLogitBytes) != cudaSuccess)
      return AHAKV_ERR_CUDA;
    configured[dev] = kStepMaxLogitBytes;
  }
  const Shape& shape = pl;
  step_slots_kernel<T, D, kG><<<pl.B * pl.Hkv, kStepThreads, smem, st>>>(
      (const T*)q, (const T*)k_new, (const T*)v_new, (T*)k, (T*)v, score, pos, free_slot, shape,
      pl.lambda[0] * 1.4426950408889634, new_pos);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

template <typename T, int D>
ahakv_status launch_slots_g(const Plan& pl, const void* q, const void* k_new, const void* v_new, void* k, void* v,
                            float* score, int32_t* pos, int32_t* free_slot, int new_pos, cudaStream_t st) {
  switch (pl.G) {
    case 1: return launch_slots_as<T, D, 1>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 2: return launch_slots_as<T, D, 2>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 3: return launch_slots_as<T, D, 3>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 4: return launch_slots_as<T, D, 4>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 5: return launch_slots_as<T, D, 5>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 6: return launch_slots_as<T, D, 6>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 7: return launch_slots_as<T, D, 7>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 8: return launch_slots_as<T, D, 8>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 12: return launch_slots_as<T, D, 12>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case 16: return launch_slots_as<T, D, 16>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    default: return AHAKV_ERR_UNSUPPORTED;
  }
}

template <typename T, int D>
ahakv_status launch_step_g(const Plan& pl, const void* q, const void* k, const float* prev, float* score, cudaStream_t st) {
  switch (pl.G) {
    case 1: return launch_step_as<T, D, 1>(pl, q, k, prev, score, st);
    case 2: return launch_step_as<T, D, 2>(pl, q, k, prev, score, st);
    case 3: return launch_step_as<T, D, 3>(pl, q, k, prev, score, st);
    case 4: return launch_step_as<T, D, 4>(pl, q, k, prev, score, st);
    case 5: return launch_step_as<T, D, 5>(pl, q, k, prev, score, st);
    case 6: return launch_step_as<T, D, 6>(pl, q, k, prev, score, st);
    case 7: return launch_step_as<T, D, 7>(pl, q, k, prev, score, st);
    case 8: return launch_step_as<T, D, 8>(pl, q, k, prev, score, st);
    case 12: return launch_step_as<T, D, 12>(pl, q, k, prev, score, st);
    case 16: return launch_step_as<T, D, 16>(pl, q, k, prev, score, st);
    default: return AHAKV_ERR_UNSUPPORTED;
  }
}

// ---- in-place compaction ------------------------------------------------------------------------------------------
constexpr int kMoveThreads = 512;
constexpr int kMoveBatchBytes = 96 * 1024;      // staged per batch: K rows, V rows (and scores)

__global__ void __launch_bounds__(kMoveThreads) compact_inplace_kernel(char* __restrict__ k, char* __restrict__ v,
                                                                       float* __restrict__ score,
                                                                       const int32_t* __restrict__ kept, const Shape pl,
                                                                       const int rows_per_batch) {
  extern __shared__ __align__(16) char stage[];
  __shared__ int first_moved;
  const int unit = blockIdx.x, n_keep = pl.n_keep;
  const long long b = unit / pl.Hkv, h = unit % pl.Hkv;
  const int32_t* idx = kept + (size_t)unit * n_keep;
  const int row_bytes = pl.d * pl.es, lanes = row_bytes / 16;
  char* kb = k + (b * pl.ks[0] + h * pl.ks[1]) * pl.es;
  char* vb = v + (b * pl.vs[0] + h * pl.vs[1]) * pl.es;
  const long long ktok = pl.ks[2] * pl.es, vtok = pl.vs[2] * pl.es;
  float* sc = score ? score + (size_t)unit * pl.n : nullptr;

  // rows before the first evicted index stay where they are
  if (threadIdx.x == 0) first_moved = n_keep;
  __syncthreads();
  for (int t = threadIdx.x; t < n_keep; t += kMoveThreads)
    if (idx[t] != t) { atomicMin(&first_moved, t); break; }       // ascending indices: the thread's first is its smallest
  __syncthreads();
  const int t_begin = first_moved;

  uint4* ks = reinterpret_cast<uint4*>(stage);
  uint4* vs = ks + (size_t)rows_per_batch * lanes;
  float* ss = reinterpret_cast<float*>(vs + (size_t)rows_per_batch * lanes);
  for (int t0 = t_begin; t0 < n_keep; t0 += rows_per_batch) {
    const int rows = min(rows_per_batch, n_keep - t0), chunks = rows * lanes;
    for (int c = threadIdx.x; c < chunks; c += kMoveThreads) {
      const int t = c / lanes, sub = c % lanes;
      const long long j = idx[t0 + t];
      ks[c] = *reinterpret_cast<const uint4*>(kb + j * ktok + sub * 16);
      vs[c] = *reinterpret_cast<const uint4*>(vb + j * vtok + sub * 16);
    }
    if (sc)
      for (int t = threadIdx.x; t < rows; t += kMoveThreads) ss[t] = sc[idx[t0 + t]];
    __syncthreads();                             // every row of the batch has been read
    for (int c = threadIdx.x; c < chunks; c += kMoveThreads) {
      const int t = c / lanes, sub = c % lanes;
      *reinterpret_cast<uint4*>(kb + (long long)(t0 + t) * ktok + sub * 16) = ks[c];
      *reinterpret_cast<uint4*>(vb + (long long)(t0 + t) * vtok + sub * 16) = vs[c];
    }
    if (sc)
      for (int t = threadIdx.x; t < rows; t += kMoveThreads) sc[t0 + t] = ss[t];
    __syncthreads();                             // the staging area is free, and later batches read rows written by none
  }
}

}  // namespace

bool step_score_fits(const Plan& pl) {
  if (pl.r != 1 || pl.G > kStepMaxG || (size_t)pl.G * pl.n * sizeof(float) > kStepMaxLogitBytes) return false;
  return pl.G <= 8 || pl.G == 12 || pl.G == 16;
}

ahakv_status launch_step_score(const Plan& pl, const void* q, const void* k, const float* prev, float* score,
                               cudaStream_t st) {
  const bool d64 = pl.d == 64;
  switch (pl.dtype) {
    case AHAKV_F32: return d64 ? launch_step_g<float, 64>(pl, q, k, prev, score, st) : launch_step_g<float, 128>(pl, q, k, prev, score, st);
    case AHAKV_F16: return d64 ? launch_step_g<__half, 64>(pl, q, k, prev, score, st) : launch_step_g<__half, 128>(pl, q, k, prev, score, st);
    default: return d64 ? launch_step_g<__nv_bfloat16, 64>(pl, q, k, prev, score, st)
                        : launch_step_g<__nv_bfloat16, 128>(pl, q, k, prev, score, st);
  }
}

ahakv_status launch_step_slots(const Plan& pl, const void* q, const void* k_new, const void* v_new, void* k, void* v,
                               float* score, int32_t* pos, int32_t* free_slot, int new_pos, cudaStream_t st) {
  const bool d64 = pl.d == 64;
  switch (pl.dtype) {
    case AHAKV_F32:
      return d64 ? launch_slots_g<float, 64>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st)
                 : launch_slots_g<float, 128>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    case AHAKV_F16:
      return d64 ? launch_slots_g<__half, 64>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st)
                 : launch_slots_g<__half, 128>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
    default:
      return d64 ? launch_slots_g<__nv_bfloat16, 64>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st)
                 : launch_slots_g<__nv_bfloat16, 128>(pl, q, k_new, v_new, k, v, score, pos, free_slot, new_pos, st);
  }
}

ahakv_status launch_compact_inplace(const Plan& pl, void* k, void* v, float* score, const int32_t* kept_idx,
                                    cudaStream_t st) {
  const int row_bytes = pl.d * pl.es;
  const int per_row = 2 * row_bytes + (int)sizeof(float);
  int rows_per_batch = kMoveBatchBytes / per_row;
  rows_per_batch -= rows_per_batch % 4;          // keeps the staged scores 16-byte aligned behind the rows
  constexpr int kMaxDevices = 64;
  static bool configured[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AHAKV_ERR_CUDA;
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(compact_inplace_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMoveBatchBytes) != cudaSuccess)
      return AHAKV_ERR_CUDA;
    configured[dev] = true;
  }
  const Shape& shape = pl;
  compact_inplace_kernel<<<pl.B * pl.Hkv, kMoveThreads, (size_t)rows_per_batch * per_row, st>>>(
      (char*)k, (char*)v, score, kept_idx, shape, rows_per_batch);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace ahakv
