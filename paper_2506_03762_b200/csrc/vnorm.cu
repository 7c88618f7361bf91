// nu_j = |V_j|^2 (Section 4.3): one coalesced 128-bit streaming pass over V.
// LANES consecutive threads read one row (16 bytes each), square and add in FP32
// and fold with a fixed shuffle tree; each thread keeps several rows in flight.
#include "ahakv_internal.cuh"

namespace ahakv {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsInFlight = 4;

__device__ __forceinline__ uint4 ld_stream(const void* p) {  // read once: do not keep in L1, evict first from L2
  uint4 v;
  asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

template <typename T, int LANES>
__global__ void __launch_bounds__(kThreads) vnorm_kernel(const T* __restrict__ v, float* __restrict__ nu, const Shape pl) {
  constexpr int V = Vec16<T>::N;
  const long long total_rows = (long long)pl.B * pl.Hkv * pl.n;
  const long long groups = (long long)gridDim.x * (kThreads / LANES);
  const long long group = (long long)blockIdx.x * (kThreads / LANES) + threadIdx.x / LANES;
  const int lane = threadIdx.x % LANES;
  // The loop bound is taken from the warp's first group so that all 32 lanes stay in the shuffles.
  const long long warp_first = group - (threadIdx.x % 32) / LANES;
  for (long long base = group; base - (group - warp_first) < total_rows; base += groups * kRowsInFlight) {
    uint4 u[kRowsInFlight];
    bool ok[kRowsInFlight];
#pragma unroll
    for (int t = 0; t < kRowsInFlight; ++t) {
      const long long row = base + t * groups;
      ok[t] = row < total_rows;
      if (ok[t]) {
        const long long unit = row / pl.n, j = row % pl.n;
        const long long b = unit / pl.Hkv, h = unit % pl.Hkv;
        u[t] = ld_stream(v + b * pl.vs[0] + h * pl.vs[1] + j * pl.vs[2] + lane * V);
      } else {
        u[t] = make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int t = 0; t < kRowsInFlight; ++t) {
      float f[V];
      Vec16<T>::widen(u[t], f);
      float s = 0.f;
#pragma unroll
      for (int c = 0; c < V; ++c) s = fmaf(f[c], f[c], s);
#pragma unroll
      for (int o = LANES / 2; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0 && ok[t]) nu[base + t * groups] = s;
    }
  }
}

template <typename T, int LANES>
ahakv_status run(const Plan& pl, const void* v, float* nu, cudaStream_t st) {
  const long long total_rows = (long long)pl.B * pl.Hkv * pl.n;
  const long long rows_per_block = (long long)(kThreads / LANES) * kRowsInFlight;
  long long blocks = (total_rows + rows_per_block - 1) / rows_per_block;
  const long long cap = 148LL * 8 * 4;
  if (blocks > cap) blocks = cap;
  vnorm_kernel<T, LANES><<<(unsigned)blocks, kThreads, 0, st>>>((const T*)v, nu, pl);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace

ahakv_status launch_vnorm(const Plan& pl, const void* v, float* nu, cudaStream_t st) {
  const int lanes = pl.d * pl.es / 16;
  if (pl.dtype == AHAKV_F32) return lanes == 16 ? run<float, 16>(pl, v, nu, st) : run<float, 32>(pl, v, nu, st);
  if (pl.dtype == AHAKV_F16) return lanes == 8 ? run<__half, 8>(pl, v, nu, st) : run<__half, 16>(pl, v, nu, st);
  return lanes == 8 ? run<__nv_bfloat16, 8>(pl, v, nu, st) : run<__nv_bfloat16, 16>(pl, v, nu, st);
}

}  // namespace ahakv
