// Optional stage timing with CUDA events on the caller's stream.
#include <mutex>

#include "ahakv_internal.cuh"

namespace ahakv {
namespace {

constexpr int kMarks = AHAKV_N_STAGES + 1;
std::mutex g_mu;
bool g_on = false;
cudaEvent_t g_ev[AHAKV_PROFILE_MAX_CALLS][kMarks];
int g_next = 0;      // next slot to use
int g_count = 0;     // slots filled since the last read

}  // namespace

int profile_begin_call(cudaStream_t) {
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_on) return -1;
  const int slot = g_next;
  g_next = (g_next + 1) % AHAKV_PROFILE_MAX_CALLS;
  if (g_count < AHAKV_PROFILE_MAX_CALLS) ++g_count;
  return slot;
}

void profile_mark(int slot, int boundary, cudaStream_t st) {
  if (slot < 0) return;
  cudaEventRecord(g_ev[slot][boundary], st);
}

}  // namespace ahakv

using namespace ahakv;

extern "C" {

ahakv_status ahakv_profile_enable(int on) {
  std::lock_guard<std::mutex> lk(g_mu);
  if ((on != 0) == g_on) {
    g_next = g_count = 0;
    return AHAKV_OK;
  }
  if (on) {
    for (int s = 0; s < AHAKV_PROFILE_MAX_CALLS; ++s)
      for (int m = 0; m < kMarks; ++m)
        if (cudaEventCreate(&g_ev[s][m]) != cudaSuccess) return AHAKV_ERR_CUDA;
  } else {
    cudaDeviceSynchronize();
    for (int s = 0; s < AHAKV_PROFILE_MAX_CALLS; ++s)
      for (int m = 0; m < kMarks; ++m) cudaEventDestroy(g_ev[s][m]);
  }
  g_on = on != 0;
  g_next = g_count = 0;
  return AHAKV_OK;
}

int64_t ahakv_profile_read(double* ms) {
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_on || !ms) return -1;
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  for (int t = 0; t < AHAKV_N_STAGES; ++t) ms[t] = 0.0;
  const int count = g_count;
  for (int c = 0; c < count; ++c) {
    const int slot = ((g_next - 1 - c) % AHAKV_PROFILE_MAX_CALLS + AHAKV_PROFILE_MAX_CALLS) % AHAKV_PROFILE_MAX_CALLS;
    for (int t = 0; t < AHAKV_N_STAGES; ++t) {
      float e = 0.f;
      if (cudaEventElapsedTime(&e, g_ev[slot][t], g_ev[slot][t + 1]) == cudaSuccess) ms[t] += (double)e;
    }
  }
  g_next = g_count = 0;
  return count;
}

const char* ahakv_stage_name(int stage) {
  static const char* names[AHAKV_N_STAGES] = {"score", "vnorm", "refine", "select", "compact"};
  return (stage >= 0 && stage < AHAKV_N_STAGES) ? names[stage] : "?";
}

}  // extern "C"
