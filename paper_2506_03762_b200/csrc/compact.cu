// Compaction (Algorithm 1, generation phase: K <- K_S, V <- V_S): a vectorised
// gather.  LANES consecutive threads move one kept row of K and of V, 16 bytes
// each, from its strided source to the dense output; lane 0 also carries the
// row's score.  Pure byte movement: the element type never matters.
#include "ahakv_internal.cuh"

namespace ahakv {
namespace {

constexpr int kThreads = 256;

template <int LANES>
__global__ void __launch_bounds__(kThreads) compact_kernel(const char* __restrict__ k, const char* __restrict__ v,
                                                           const float* __restrict__ score,
                                                           const int32_t* __restrict__ kept, char* __restrict__ k_out,
                                                           char* __restrict__ v_out, float* __restrict__ score_out,
                                                           const Shape pl) {
  const long long total = (long long)pl.B * pl.Hkv * pl.n_keep;
  const long long stride = (long long)gridDim.x * (kThreads / LANES);
  const int lane = threadIdx.x % LANES;
  for (long long row = (long long)blockIdx.x * (kThreads / LANES) + threadIdx.x / LANES; row < total; row += stride) {
    const long long unit = row / pl.n_keep;
    const long long b = unit / pl.Hkv, h = unit % pl.Hkv;
    const int j = kept[row];
    if (j < 0) continue;                       // a head with a budget of its own keeps fewer rows than the stride
    const long long ksrc = (b * pl.ks[0] + h * pl.ks[1] + (long long)j * pl.ks[2]) * pl.es + lane * 16;
    const long long vsrc = (b * pl.vs[0] + h * pl.vs[1] + (long long)j * pl.vs[2]) * pl.es + lane * 16;
    const long long dst = row * (long long)(LANES * 16) + lane * 16;
    const uint4 kv = *reinterpret_cast<const uint4*>(k + ksrc);
    const uint4 vv = *reinterpret_cast<const uint4*>(v + vsrc);
    *reinterpret_cast<uint4*>(k_out + dst) = kv;
    *reinterpret_cast<uint4*>(v_out + dst) = vv;
    if (score_out && lane == 0) score_out[row] = score[unit * pl.n + j];
  }
}

template <int LANES>
ahakv_status run(const Plan& pl, const void* k, const void* v, const float* score, const int32_t* kept, void* k_out,
                 void* v_out, float* score_out, cudaStream_t st) {
  const long long total = (long long)pl.B * pl.Hkv * pl.n_keep;
  const long long rows_per_block = kThreads / LANES;
  long long blocks = (total + rows_per_block - 1) / rows_per_block;
  const long long cap = 148LL * 8 * 8;
  if (blocks > cap) blocks = cap;
  compact_kernel<LANES><<<(unsigned)blocks, kThreads, 0, st>>>((const char*)k, (const char*)v, score, kept,
                                                               (char*)k_out, (char*)v_out, score_out, pl);
  count_launch();
  return cuda_ok(cudaGetLastError());
}

}  // namespace

ahakv_status launch_compact(const Plan& pl, const void* k, const void* v, const float* score,
                            const int32_t* kept_idx, void* k_out, void* v_out, float* score_out,
                            cudaStream_t st) {
  switch (pl.d * pl.es / 16) {
    case 8: return run<8>(pl, k, v, score, kept_idx, k_out, v_out, score_out, st);
    case 16: return run<16>(pl, k, v, score, kept_idx, k_out, v_out, score_out, st);
    default: return run<32>(pl, k, v, score, kept_idx, k_out, v_out, score_out, st);
  }
}

}  // namespace ahakv
