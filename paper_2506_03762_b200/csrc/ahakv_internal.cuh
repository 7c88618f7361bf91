// Internal declarations shared by the translation units of libahakv.so.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ahakv.h"

namespace ahakv {

constexpr int kMaxRows = 256;   // G * r, the stacked observation rows of one KV head
constexpr int kKeyTile = 128;   // keys per scoring tile
constexpr float kLog2e = 1.4426950408889634f;

// Per observation row i: c[i] = lambda_i * log2(e), so that e^{lambda w} = 2^{c w}.
struct RowScale {
  float c[kMaxRows];
};

// The sizes and strides of a call: the part of the plan that the small kernels take by value.
struct Shape {
  int B, Hq, Hkv, G, d, n, r, Br, Bud, Bs, n_keep, dtype, es, pool;
  unsigned flags;
  long long n_total;
  int R;          // G * r
  int n_blk;      // ceil(n / kKeyTile)
  int group_max;  // pool the query heads of a KV head by maximum instead of mean (and G > 1)
  long long qs[3], ks[3], vs[3];  // element strides: batch, head, token
};

// Everything the host derives from ahakv_params once per call.
struct Plan : Shape {
  int n_rb;       // row blocks of 128 stacked rows (tensor-core path)
  int heads_per_rb;  // query heads per row block (tensor-core path)
  bool use_tc;    // tensor-core scoring path applies
  RowScale rows;
  double lambda[kMaxRows];   // lambda_i itself, in double (the float32 path scales its logits in double)
  int last[kMaxRows];        // per observation row: the last cache row it may see (n - r + i unless positions are given)
  int n_eff;                 // last[r - 1] + 1: keys beyond are seen by no row
  // workspace layout, byte offsets
  size_t off_status, off_sync, off_sraw, off_nu, off_partial, off_final, off_score, ws_total;
};

// plan.cu
// `obs_pos` (nullable, host, r ascending logical positions) places the observation rows; by default they are the
// last r positions.
ahakv_status make_plan(const ahakv_params* p, Plan* plan, const int64_t* obs_pos = nullptr);
void count_launch(int n = 1);

// Launchers.  Each returns AHAKV_OK or AHAKV_ERR_CUDA and queues work on `st` only.
ahakv_status launch_score_simt(const Plan& pl, const void* q, const void* k, float* s_raw, float2* partial,
                               float* final_off, cudaStream_t st);
// Also streams V and writes nu when the value prior is on (v and nu non-null).
ahakv_status launch_score_tc(const Plan& pl, const void* q, const void* k, const void* v, float* s_raw, float* nu,
                             float2* partial, int* counters, int* status, cudaStream_t st);
bool score_tc_available();
void score_tc_test_hooks(long long wait_ns, int withhold);   // see ahakv_test_set_wait
// The generation phase one token at a time (decode.cu): the score update of one new query per head without
// scratch memory, and compaction in place.
bool step_score_fits(const Plan& pl);
ahakv_status launch_step_slots(const Plan& pl, const void* q, const void* k_new, const void* v_new, void* k, void* v,
                               float* score, int32_t* pos, int32_t* free_slot, int new_pos, cudaStream_t st);
ahakv_status launch_step_score(const Plan& pl, const void* q, const void* k, const float* prev, float* score,
                               cudaStream_t st);
ahakv_status launch_compact_inplace(const Plan& pl, void* k, void* v, float* score, const int32_t* kept_idx,
                                    cudaStream_t st);
// Row entropy of the SG-softmax (entropy.cu): out [B, Hq, r]; `scratch` of entropy_scratch_bytes().
size_t entropy_scratch_bytes(const Plan& pl);
ahakv_status launch_entropy(const Plan& pl, const void* q, const void* k, void* scratch, float* out, cudaStream_t st);
ahakv_status launch_vnorm(const Plan& pl, const void* v, float* nu, cudaStream_t st);
// `slots` partial scores per head (row blocks, or query heads when pooling by maximum) are combined here.
ahakv_status launch_refine(const Plan& pl, const float* s_raw, const float* nu, const float* score_prev,
                           float* score, int slots, cudaStream_t st);
ahakv_status launch_select(const Plan& pl, const float* score, int32_t* kept_idx, const int32_t* budgets,
                           cudaStream_t st);
bool refine_select_fits(const Plan& pl);
ahakv_status launch_refine_select(const Plan& pl, const float* s_raw, const float* nu, const float* score_prev,
                                  float* score, int32_t* kept_idx, int slots, const int32_t* budgets,
                                  cudaStream_t st);
ahakv_status launch_compact(const Plan& pl, const void* k, const void* v, const float* score,
                            const int32_t* kept_idx, void* k_out, void* v_out, float* score_out,
                            cudaStream_t st);

// profile.cu: event marks around the stages of a call (no-ops unless profiling is enabled).
int profile_begin_call(cudaStream_t st);             // returns a slot, or -1
void profile_mark(int slot, int boundary, cudaStream_t st);   // boundary b closes stage b-1, opens stage b

inline ahakv_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? AHAKV_OK : AHAKV_ERR_CUDA; }

// ---- device helpers ---------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__half>(__half x) { return __half2float(x); }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

// 16 bytes of T widened to float.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void widen(const uint4& u, float* f) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y);
    f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
  }
};
template <> struct Vec16<__half> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void widen(const uint4& u, float* f) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&w[t]));
      f[2 * t] = p.x; f[2 * t + 1] = p.y;
    }
  }
};
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void widen(const uint4& u, float* f) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {  // a bfloat16 is the high half of a float
      f[2 * t] = __uint_as_float(w[t] << 16);
      f[2 * t + 1] = __uint_as_float(w[t] & 0xffff0000u);
    }
  }
};

__device__ __forceinline__ float fast_exp2(float x) {  // 2 ulp over the whole range; 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace ahakv
