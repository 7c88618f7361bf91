// Row entropy of the SG-softmax (Eq. 6): H_i = - sum_j a_ij ln a_ij for every observation row of every query
// head.  A diagnostic next to the score: Eq. 10 predicts E[H_i] = ln i - lambda^2 d / 2 and Eq. 12 chooses lambda
// so that it equals ln(budget); this lets a caller check that on real activations, or tune lambda with it.
//
// With x_j = c w_j (log2 units), M a shift, Z = sum 2^{x_j - M} and T = sum 2^{x_j - M} (x_j - M):
//   H = ln 2 (log2 Z - T / Z).
// Per 128-key tile and row the triple (M, Z, T) is formed and written out, and a second kernel folds the tiles in
// order.  16-bit inputs: the tile's logits come from warp-level m16n8k16 products, 32 rows a warp, and every thread
// folds its two keys of a row into a running triple (entropy_tiles_mma).  float32 inputs: one thread owns one key
// (as in the FP32-pipe scoring kernels), logits in double, the triple formed by warp shuffles (entropy_tiles).
// Fixed reduction order either way, so the result is reproducible bit for bit.
#include <type_traits>

#include "ahakv_internal.cuh"
#include "mma_sync.cuh"

namespace ahakv {
namespace {

constexpr int kThreads = 128;

template <typename T> using Acc = typename std::conditional<std::is_same<T, float>::value, double, float>::type;
template <typename A> struct RowTable {
  A c[kMaxRows];
  int last[kMaxRows];
};

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) entropy_tiles(const T* __restrict__ q, const T* __restrict__ k,
                                                          float4* __restrict__ partial, const Shape pl,
                                                          const RowTable<Acc<T>> rt) {
  using A = Acc<T>;
  constexpr int V = Vec16<T>::N;
  extern __shared__ __align__(16) float smem[];
  float* qsm = smem;                                               // [r][D]
  float4* wst = reinterpret_cast<float4*>(smem + pl.r * D);        // [4][r]
  const int uq = blockIdx.y, b = uq / pl.Hq, hq = uq % pl.Hq, h = hq / pl.G, blk = blockIdx.x;
  const int j = blk * kKeyTile + threadIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int t = threadIdx.x; t < pl.r * (D / V); t += kThreads) {
    const int i = t / (D / V), cv = t % (D / V);
    const T* row = q + (long long)b * pl.qs[0] + (long long)hq * pl.qs[1] + (long long)i * pl.qs[2];
    Vec16<T>::widen(*reinterpret_cast<const uint4*>(row + cv * V), qsm + i * D + cv * V);
  }
  float kreg[D];
  const bool valid = j < pl.n;
  if (valid) {
    const T* row = k + (long long)b * pl.ks[0] + (long long)h * pl.ks[1] + (long long)j * pl.ks[2];
#pragma unroll
    for (int cv = 0; cv < D / V; ++cv) Vec16<T>::widen(*reinterpret_cast<const uint4*>(row + cv * V), kreg + cv * V);
  } else {
#pragma unroll
    for (int c = 0; c < D; ++c) kreg[c] = 0.f;
  }
  __syncthreads();
  for (int i = 0; i < pl.r; ++i) {
    const bool vis = valid && j <= rt.last[i];
    A a0 = 0, a1 = 0, a2 = 0, a3 = 0;
#pragma unroll
    for (int c = 0; c < D; c += 4) {
      const float4 qv = *reinterpret_cast<const float4*>(qsm + i * D + c);
      a0 = fma((A)qv.x, (A)kreg[c], a0);
      a1 = fma((A)qv.y, (A)kreg[c + 1], a1);
      a2 = fma((A)qv.z, (A)kreg[c + 2], a2);
      a3 = fma((A)qv.w, (A)kreg[c + 3], a3);
    }
    const A x = vis ? ((a0 + a1) + (a2 + a3)) * rt.c[i] : (A)-INFINITY;
    float m = (float)x;
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float dx = vis ? (float)(x - (A)m) : 0.f;               // <= 0 up to the rounding of the shift
    float z = vis ? fast_exp2(dx) : 0.f, tt = z * dx;
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      z += __shfl_xor_sync(0xffffffffu, z, o);
      tt += __shfl_xor_sync(0xffffffffu, tt, o);
    }
    if (lane == 0) wst[warp * pl.r + i] = make_float4(m, z, tt, 0.f);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < pl.r; i += kThreads) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) M = fmaxf(M, wst[w * pl.r + i].x);
    float Z = 0.f, Tt = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
      const float4 p = wst[w * pl.r + i];
      if (p.y > 0.f) {
        const float s = fast_exp2(p.x - M);
        Z += p.y * s;
        Tt += (p.z + p.y * (p.x - M)) * s;
      }
    }
    partial[((size_t)uq * pl.n_blk + blk) * pl.r + i] = make_float4(M, Z, Tt, 0.f);
  }
}

// (M, Z, T) of a set of keys folded with two more keys x0, x1 (v0, v1: visible).
__device__ __forceinline__ void fold_pair(float& m, float& z, float& t, float x0, float x1, bool v0, bool v1) {
  const float mx = fmaxf(v0 ? x0 : -INFINITY, v1 ? x1 : -INFINITY);
  if (mx == -INFINITY) return;
  const float mn = fmaxf(m, mx);
  if (z > 0.f) {
    const float s = fast_exp2(m - mn);
    t = (t + z * (m - mn)) * s;
    z *= s;
  }
  m = mn;
  if (v0) { const float dx = x0 - mn, e = fast_exp2(dx); z += e; t += e * dx; }
  if (v1) { const float dx = x1 - mn, e = fast_exp2(dx); z += e; t += e * dx; }
}
// Two triples of disjoint key sets into one (the first argument), the first set's terms first.
__device__ __forceinline__ void fold_triples(float& m, float& z, float& t, float m2, float z2, float t2) {
  const float mn = fmaxf(m, m2);
  float zz = 0.f, tt = 0.f;
  if (z > 0.f) { const float s = fast_exp2(m - mn); zz += z * s; tt += (t + z * (m - mn)) * s; }
  if (z2 > 0.f) { const float s = fast_exp2(m2 - mn); zz += z2 * s; tt += (t2 + z2 * (m2 - mn)) * s; }
  m = mn; z = zz; t = tt;
}

// 16-bit inputs.  One CTA per (query head, 128-key tile), four warps; a warp takes the observation rows in blocks of
// 32 (two 16-row products side by side) and walks the tile's sixteen 8-key columns once per block, reading the keys
// straight from global memory (the tile stays in L1 for the other warps).  Operands are fed as in mma_sync.cuh: each
// thread a contiguous quarter of its row.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) entropy_tiles_mma(const T* __restrict__ q, const T* __restrict__ k,
                                                              float4* __restrict__ partial, const Shape pl,
                                                              const RowTable<float> rt) {
  constexpr int CH = D / 4, W = CH / 2, Q4 = CH / 8;
  const int uq = blockIdx.y, b = uq / pl.Hq, hq = uq % pl.Hq, h = hq / pl.G, blk = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, grp = lane >> 2, tig = lane & 3;
  const T* qbase = q + (long long)b * pl.qs[0] + (long long)hq * pl.qs[1] + CH * tig;
  const T* kbase = k + (long long)b * pl.ks[0] + (long long)h * pl.ks[1] + CH * tig;
  const int j_tile = blk * kKeyTile;
  for (int i0 = warp * 32; i0 < pl.r; i0 += (kThreads / 32) * 32) {
    // rows i0 + grp, + 8 (first product) and i0 + 16 + grp, + 8 (second)
    uint32_t a[2][2][W];
    int row[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int i = i0 + 16 * mt + 8 * hf + grp;
        row[mt][hf] = i;
#pragma unroll
        for (int t = 0; t < Q4; ++t) {
          const uint4 u = i < pl.r ? *reinterpret_cast<const uint4*>(qbase + (long long)i * pl.qs[2] + 8 * t) : make_uint4(0, 0, 0, 0);
          a[mt][hf][4 * t] = u.x; a[mt][hf][4 * t + 1] = u.y; a[mt][hf][4 * t + 2] = u.z; a[mt][hf][4 * t + 3] = u.w;
        }
      }
    float m[2][2], z[2][2], tt[2][2], c[2][2];
    int last[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        m[mt][hf] = -INFINITY; z[mt][hf] = 0.f; tt[mt][hf] = 0.f;
        const int i = row[mt][hf] < pl.r ? row[mt][hf] : 0;
        c[mt][hf] = rt.c[i];
        last[mt][hf] = row[mt][hf] < pl.r ? rt.last[i] : -1;
      }
#pragma unroll 2
    for (int nt = 0; nt < kKeyTile / 8; ++nt) {
      const int jk = j_tile + 8 * nt + grp;                       // the key this thread loads
      uint4 kw[Q4];
#pragma unroll
      for (int t = 0; t < Q4; ++t)
        kw[t] = jk < pl.n ? *reinterpret_cast<const uint4*>(kbase + (long long)jk * pl.ks[2] + 8 * t) : make_uint4(0, 0, 0, 0);
      float acc[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;
#pragma unroll
        for (int t = 0; t < Q4; ++t) {
          Mma16816<T>::run(acc[mt], a[mt][0][4 * t], a[mt][1][4 * t], a[mt][0][4 * t + 1], a[mt][1][4 * t + 1], kw[t].x, kw[t].y);
          Mma16816<T>::run(acc[mt], a[mt][0][4 * t + 2], a[mt][1][4 * t + 2], a[mt][0][4 * t + 3], a[mt][1][4 * t + 3], kw[t].z, kw[t].w);
        }
      }
      const int j0 = j_tile + 8 * nt + 2 * tig;                  // the keys this thread's results belong to: j0, j0 + 1
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int lim = min(last[mt][hf], pl.n - 1);
          fold_pair(m[mt][hf], z[mt][hf], tt[mt][hf], acc[mt][2 * hf] * c[mt][hf], acc[mt][2 * hf + 1] * c[mt][hf],
                    j0 <= lim, j0 + 1 <= lim);
        }
    }
    // the four threads of a group hold the four key classes (mod 8) of their rows: fold them in thread order
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        float M = m[mt][hf], Z = z[mt][hf], Tt = tt[mt][hf];
#pragma unroll
        for (int o = 1; o <= 2; o <<= 1) {
          const float m2 = __shfl_xor_sync(0xffffffffu, M, o), z2 = __shfl_xor_sync(0xffffffffu, Z, o),
                      t2 = __shfl_xor_sync(0xffffffffu, Tt, o);
          // both partners must add in the same order: the lower thread's set first
          if (lane & o) { float mm = m2, zz = z2, t3 = t2; fold_triples(mm, zz, t3, M, Z, Tt); M = mm; Z = zz; Tt = t3; }
          else fold_triples(M, Z, Tt, m2, z2, t2);
        }
        if (tig == 0 && row[mt][hf] < pl.r)
          partial[((size_t)uq * pl.n_blk + blk) * pl.r + row[mt][hf]] = make_float4(M, Z, Tt, 0.f);
      }
  }
}

__global__ void entropy_merge(const float4* __restrict__ partial, float* __restrict__ out, const Shape pl) {
  const int uq = blockIdx.x;
  for (int i = threadIdx.x; i < pl.r; i += blockDim.x) {
    const float4* p = partial + (size_t)uq * pl.n_blk * pl.r + i;
    float M = -INFINITY;
    for (int t = 0; t < pl.n_blk; ++t) M = fmaxf(M, p[(size_t)t * pl.r].x);
    float Z = 0.f, Tt = 0.f;
    for (int t = 0; t < pl.n_blk; ++t) {
      const float4 e = p[(size_t)t * pl.r];
      if (e.y > 0.f) {
        const float s = fast_exp2(e.x - M);
        Z += e.y * s;
        Tt += (e.z + e.y * (e.x - M)) * s;
      }
    }
    out[(size_t)uq * pl.r + i] = 0.6931471805599453f * (log2f(Z) - Tt / Z);
  }
}

template <typename T, int D>
ahakv_status run_mma(const Plan& pl, const void* q, const void* k, float4* partial, float* out, cudaStream_t st) {
  RowTable<float> rt;
  for (int i = 0; i < kMaxRows; ++i) {
    rt.c[i] = i < pl.r ? (float)(pl.lambda[i] * 1.4426950408889634) : 0.f;
    rt.last[i] = pl.last[i];
  }
  const Shape& shape = pl;
  entropy_tiles_mma<T, D><<<dim3(pl.n_blk, pl.B * pl.Hq), kThreads, 0, st>>>((const T*)q, (const T*)k, partial, shape, rt);
  entropy_merge<<<pl.B * pl.Hq, 256, 0, st>>>(partial, out, shape);
  count_launch(2);
  return cuda_ok(cudaGetLastError());
}

template <typename T, int D>
ahakv_status run(const Plan& pl, const void* q, const void* k, float4* partial, float* out, cudaStream_t st) {
  RowTable<Acc<T>> rt;
  for (int i = 0; i < kMaxRows; ++i) {
    rt.c[i] = i < pl.r ? (Acc<T>)(pl.lambda[i] * 1.4426950408889634) : (Acc<T>)0;
    rt.last[i] = pl.last[i];
  }
  const size_t smem = (size_t)pl.r * D * sizeof(float) + (size_t)(kThreads / 32) * pl.r * sizeof(float4);
  if (cudaFuncSetAttribute(entropy_tiles<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return AHAKV_ERR_CUDA;
  const Shape& shape = pl;
  entropy_tiles<T, D><<<dim3(pl.n_blk, pl.B * pl.Hq), kThreads, smem, st>>>((const T*)q, (const T*)k, partial, shape, rt);
  entropy_merge<<<pl.B * pl.Hq, 256, 0, st>>>(partial, out, shape);
  count_launch(2);
  return cuda_ok(cudaGetLastError());
}

}  // namespace

size_t entropy_scratch_bytes(const Plan& pl) {
  return ((size_t)pl.B * pl.Hq * pl.n_blk * pl.r * sizeof(float4) + 255) / 256 * 256;
}

ahakv_status launch_entropy(const Plan& pl, const void* q, const void* k, void* scratch, float* out, cudaStream_t st) {
  float4* partial = reinterpret_cast<float4*>(scratch);
  const bool d64 = pl.d == 64;
  switch (pl.dtype) {
    case AHAKV_F32: return d64 ? run<float, 64>(pl, q, k, partial, out, st) : run<float, 128>(pl, q, k, partial, out, st);
    case AHAKV_F16: return d64 ? run_mma<__half, 64>(pl, q, k, partial, out, st) : run_mma<__half, 128>(pl, q, k, partial, out, st);
    default: return d64 ? run_mma<__nv_bfloat16, 64>(pl, q, k, partial, out, st)
                        : run_mma<__nv_bfloat16, 128>(pl, q, k, partial, out, st);
  }
}

}  // namespace ahakv
