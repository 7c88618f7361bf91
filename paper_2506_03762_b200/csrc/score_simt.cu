// Scoring on the plain FP32 pipes: the path for float32 inputs (where a TF32
// tensor-core product would miss the 1e-5 tolerance) and for 16-bit shapes the
// tensor-core kernel does not take.
//
// One thread owns one key.  Pass 1 gives every observation row its softmax
// statistics (max and sum of 2^{c w}) per 128-key tile, a small kernel merges the
// tiles, and pass 2 recomputes the logits and adds the normalised weights of all
// rows into the key's score (Eq. 1, 5, 9).  Every reduction has a fixed order,
// so the scores are reproducible bit for bit.
//
// float32 inputs are held to 1e-5 on the scores, logits of hundreds included: an FP32
// logit near 256 is only known to 3e-5, so for them the dot product, the scale and
// the subtraction of the row's shift run in double (products of two floats are exact
// there), and only the shifted exponent, a small number, goes back to FP32 for the
// exponential.  16-bit inputs (1e-3) keep FP32 throughout.
#include <type_traits>

#include "ahakv_internal.cuh"

namespace ahakv {
namespace {

constexpr int kThreads = 128;

template <typename T, int D>
__device__ __forceinline__ void load_q_group(const T* __restrict__ q, const Shape& pl, int b, int h, float* qsm) {
  // qsm[s][c], s = g * r + i over the G query heads of KV head h
  constexpr int V = Vec16<T>::N;
  const int vec_per_row = D / V;
  for (int t = threadIdx.x; t < pl.R * vec_per_row; t += blockDim.x) {
    const int s = t / vec_per_row, cv = t % vec_per_row;
    const int g = s / pl.r, i = s % pl.r;
    const T* row = q + (long long)b * pl.qs[0] + (long long)(h * pl.G + g) * pl.qs[1] + (long long)i * pl.qs[2];
    const uint4 u = *reinterpret_cast<const uint4*>(row + cv * V);
    Vec16<T>::widen(u, qsm + s * D + cv * V);
  }
}

template <typename T, int D>
__device__ __forceinline__ void load_key(const T* __restrict__ k, const Shape& pl, int b, int h, int j, float* kreg) {
  constexpr int V = Vec16<T>::N;
  const T* row = k + (long long)b * pl.ks[0] + (long long)h * pl.ks[1] + (long long)j * pl.ks[2];
#pragma unroll
  for (int cv = 0; cv < D / V; ++cv) {
    const uint4 u = *reinterpret_cast<const uint4*>(row + cv * V);
    Vec16<T>::widen(u, kreg + cv * V);
  }
}

// The accumulator type of the logits: double for float32 inputs, float for 16-bit ones.
template <typename T> using Acc = typename std::conditional<std::is_same<T, float>::value, double, float>::type;

// Per observation row: lambda_i log2(e) in the accumulator's type, and the last cache row it may see.
template <typename A> struct RowScaleOf {
  A c[kMaxRows];
  int last[kMaxRows];
};

template <int D, typename A>
__device__ __forceinline__ A dot_row(const float* __restrict__ qrow, const float* kreg) {
  A a0 = 0, a1 = 0, a2 = 0, a3 = 0;
#pragma unroll
  for (int c = 0; c < D; c += 4) {
    const float4 qv = *reinterpret_cast<const float4*>(qrow + c);
    a0 = fma((A)qv.x, (A)kreg[c], a0);
    a1 = fma((A)qv.y, (A)kreg[c + 1], a1);
    a2 = fma((A)qv.z, (A)kreg[c + 2], a2);
    a3 = fma((A)qv.w, (A)kreg[c + 3], a3);
  }
  return (a0 + a1) + (a2 + a3);
}

// Pass 1: per (unit, key tile, stacked row) the pair (max of c*w, sum of 2^{c*w - max}).
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) simt_row_stats(const T* __restrict__ q, const T* __restrict__ k,
                                                           float2* __restrict__ partial, const Shape pl,
                                                           const RowScaleOf<Acc<T>> cs) {
  using A = Acc<T>;
  extern __shared__ __align__(16) float smem[];
  float* qsm = smem;                                            // [R][D]
  float2* wst = reinterpret_cast<float2*>(smem + pl.R * D);     // [4][R]
  const int unit = blockIdx.y, b = unit / pl.Hkv, h = unit % pl.Hkv, blk = blockIdx.x;
  const int j = blk * kKeyTile + threadIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  load_q_group<T, D>(q, pl, b, h, qsm);
  float kreg[D];
  const bool valid = j < pl.n;
  if (valid) load_key<T, D>(k, pl, b, h, j, kreg);
  else {
#pragma unroll
    for (int c = 0; c < D; ++c) kreg[c] = 0.f;
  }
  __syncthreads();
  for (int s = 0; s < pl.R; ++s) {
    const int i = s % pl.r;
    const bool vis = valid && j <= cs.last[i];
    const A x = vis ? dot_row<D, A>(qsm + s * D, kreg) * cs.c[i] : (A)-INFINITY;
    float m = (float)x;                                         // the shift is an FP32 number on either path
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float z = vis ? fast_exp2((float)(x - (A)m)) : 0.f;
#pragma unroll
    for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    if (lane == 0) wst[warp * pl.R + s] = make_float2(m, z);
  }
  __syncthreads();
  for (int s = threadIdx.x; s < pl.R; s += kThreads) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) M = fmaxf(M, wst[w * pl.R + s].x);
    float Z = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
      const float2 p = wst[w * pl.R + s];
      if (p.y > 0.f) Z += p.y * fast_exp2(p.x - M);
    }
    partial[((size_t)unit * pl.n_blk + blk) * pl.R + s] = make_float2(M, Z);
  }
}

// Merge the tiles of one unit into (max, 1 / (G * sum)) per stacked row, so that
// 2^{c w - max} times the second entry is the softmax weight divided by the group size.
__global__ void simt_merge_stats(const float2* __restrict__ partial, float2* __restrict__ final_st, const Shape pl) {
  const int unit = blockIdx.x;
  for (int s = threadIdx.x; s < pl.R; s += blockDim.x) {
    const float2* p = partial + (size_t)unit * pl.n_blk * pl.R + s;
    float M = -INFINITY;
    for (int t = 0; t < pl.n_blk; ++t) M = fmaxf(M, p[(size_t)t * pl.R].x);
    float Z = 0.f;
    for (int t = 0; t < pl.n_blk; ++t) {
      const float2 e = p[(size_t)t * pl.R];
      if (e.y > 0.f) Z += e.y * fast_exp2(e.x - M);
    }
    final_st[(size_t)unit * pl.R + s] = make_float2(M, 1.f / (Z * (float)(pl.group_max ? 1 : pl.G)));
  }
}

// Pass 2: S_j = sum over the stacked rows of 2^{c w - max} / (G * sum).
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) simt_column_sums(const T* __restrict__ q, const T* __restrict__ k,
                                                             const float2* __restrict__ final_st,
                                                             float* __restrict__ s_raw, const Shape pl,
                                                             const RowScaleOf<Acc<T>> cs) {
  using A = Acc<T>;
  extern __shared__ __align__(16) float smem[];
  float* qsm = smem;                                            // [R][D]
  float2* st = reinterpret_cast<float2*>(smem + pl.R * D);      // [R]
  const int unit = blockIdx.y, b = unit / pl.Hkv, h = unit % pl.Hkv;
  const int j = blockIdx.x * kKeyTile + threadIdx.x;
  load_q_group<T, D>(q, pl, b, h, qsm);
  for (int s = threadIdx.x; s < pl.R; s += kThreads) st[s] = final_st[(size_t)unit * pl.R + s];
  __syncthreads();
  if (j >= pl.n) return;
  float kreg[D];
  load_key<T, D>(k, pl, b, h, j, kreg);
  float acc = 0.f, best = 0.f;
  for (int s = 0; s < pl.R; ++s) {
    const int i = s % pl.r;
    if (pl.group_max && i == 0 && s > 0) {        // a query head is complete: keep the largest head's score
      best = fmaxf(best, acc);
      acc = 0.f;
    }
    if (j <= cs.last[i])
      acc = fmaf(fast_exp2((float)fma(dot_row<D, A>(qsm + s * D, kreg), cs.c[i], -(A)st[s].x)), st[s].y, acc);
  }
  s_raw[(size_t)unit * pl.n + j] = pl.group_max ? fmaxf(best, acc) : acc;
}

template <typename T, int D>
ahakv_status run(const Plan& pl, const void* q, const void* k, float* s_raw, float2* partial, float* final_off,
                 cudaStream_t st) {
  RowScaleOf<Acc<T>> cs;
  for (int i = 0; i < kMaxRows; ++i) {
    cs.c[i] = i < pl.r ? (Acc<T>)(pl.lambda[i] * 1.4426950408889634) : (Acc<T>)0;
    cs.last[i] = pl.last[i];
  }
  const size_t smem1 = (size_t)pl.R * D * sizeof(float) + (size_t)(kThreads / 32) * pl.R * sizeof(float2);
  const size_t smem2 = (size_t)pl.R * D * sizeof(float) + (size_t)pl.R * sizeof(float2);
  if (cudaFuncSetAttribute(simt_row_stats<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem1) != cudaSuccess ||
      cudaFuncSetAttribute(simt_column_sums<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess)
    return AHAKV_ERR_CUDA;
  const dim3 grid(pl.n_blk, pl.B * pl.Hkv);
  simt_row_stats<T, D><<<grid, kThreads, smem1, st>>>((const T*)q, (const T*)k, partial, pl, cs);
  float2* final_st = reinterpret_cast<float2*>(final_off);
  simt_merge_stats<<<pl.B * pl.Hkv, 256, 0, st>>>(partial, final_st, pl);
  simt_column_sums<T, D><<<grid, kThreads, smem2, st>>>((const T*)q, (const T*)k, final_st, s_raw, pl, cs);
  count_launch(3);
  return cuda_ok(cudaGetLastError());
}

}  // namespace

ahakv_status launch_score_simt(const Plan& pl, const void* q, const void* k, float* s_raw, float2* partial,
                               float* final_off, cudaStream_t st) {
  const bool d64 = pl.d == 64;
  switch (pl.dtype) {
    case AHAKV_F32:
      return d64 ? run<float, 64>(pl, q, k, s_raw, partial, final_off, st)
                 : run<float, 128>(pl, q, k, s_raw, partial, final_off, st);
    case AHAKV_F16:
      return d64 ? run<__half, 64>(pl, q, k, s_raw, partial, final_off, st)
                 : run<__half, 128>(pl, q, k, s_raw, partial, final_off, st);
    default:
      return d64 ? run<__nv_bfloat16, 64>(pl, q, k, s_raw, partial, final_off, st)
                 : run<__nv_bfloat16, 128>(pl, q, k, s_raw, partial, final_off, st);
  }
}

}  // namespace ahakv
