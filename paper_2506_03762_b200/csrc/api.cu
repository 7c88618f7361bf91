// Host side of libahakv.so: argument checking, the per-call plan, the workspace
// layout and the order in which the kernels are queued.
#include <atomic>
#include <cmath>
#include <cstring>

#include <nvtx3/nvToolsExt.h>

#include "ahakv_internal.cuh"

// A named range on the host's timeline for a profiler's trace (NVTX; costs nothing when no tool is attached): one
// around every eviction call and one around the launches of each of its phases.
namespace {
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};
}  // namespace

static_assert(sizeof(ahakv_params) == 136, "ahakv_params layout is part of the ABI");

namespace ahakv {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Eq. 12 in double on the host; outside its domain the plain 1/sqrt(d).
static double eq12(double tokens, double budget, int d) {
  const double ratio = tokens / budget;
  if (!(ratio > 1.0)) return 1.0 / std::sqrt((double)d);
  return std::sqrt(2.0 * std::log(ratio) / (double)d);
}

static bool resolve_strides(const int64_t in[3], long long out[3], long long heads, long long tokens, int d,
                            int es) {
  if (in[0] == 0 && in[1] == 0 && in[2] == 0) {
    out[2] = d;
    out[1] = tokens * d;
    out[0] = heads * tokens * d;
    return true;
  }
  const long long per16 = 16 / es;
  for (int t = 0; t < 3; ++t) {
    if (in[t] <= 0 || in[t] % per16 != 0) return false;  // rows must stay 16-byte aligned
    out[t] = in[t];
  }
  return out[2] >= d;
}

ahakv_status make_plan(const ahakv_params* p, Plan* pl, const int64_t* obs_pos) {
  if (!p || !pl) return AHAKV_ERR_INVALID_ARG;
  if (p->batch < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->n_q_heads % p->n_kv_heads != 0)
    return AHAKV_ERR_INVALID_ARG;
  if (p->head_dim != 64 && p->head_dim != 128) return AHAKV_ERR_INVALID_ARG;
  if (p->n_ctx < 1 || p->n_total < p->n_ctx) return AHAKV_ERR_INVALID_ARG;
  if (p->dtype < AHAKV_F32 || p->dtype > AHAKV_BF16) return AHAKV_ERR_INVALID_ARG;
  if (p->budget < 1 || p->recent_window < 0 || p->recent_window > p->budget) return AHAKV_ERR_INVALID_ARG;
  const int G = p->n_q_heads / p->n_kv_heads;
  if (p->obs_window < 1 || p->obs_window > p->n_ctx || (long long)p->obs_window * G > kMaxRows)
    return AHAKV_ERR_INVALID_ARG;
  if (p->scale_mode < AHAKV_SCALE_FIXED || p->scale_mode > AHAKV_SCALE_ADAPTIVE_CALL) return AHAKV_ERR_INVALID_ARG;
  if (p->scale_mode == AHAKV_SCALE_FIXED && !(p->scale > 0.f && std::isfinite(p->scale)))
    return AHAKV_ERR_INVALID_ARG;
  if (p->pool_kernel < 1 || (p->pool_kernel & 1) == 0) return AHAKV_ERR_INVALID_ARG;
  if (p->flags & ~(uint32_t)(AHAKV_FLAG_VALUE_PRIOR | AHAKV_FLAG_POOL_ZERO_PAD | AHAKV_FLAG_GROUP_MAX))
    return AHAKV_ERR_INVALID_ARG;
  if ((long long)p->batch * p->n_kv_heads > 65535LL) return AHAKV_ERR_INVALID_ARG;

  Plan& o = *pl;
  o.B = p->batch; o.Hq = p->n_q_heads; o.Hkv = p->n_kv_heads; o.G = G; o.d = p->head_dim;
  o.n = p->n_ctx; o.r = p->obs_window; o.Br = p->recent_window; o.Bud = p->budget;
  o.Bs = p->budget - p->recent_window;
  o.n_keep = p->n_ctx < p->budget ? p->n_ctx : p->budget;
  o.dtype = p->dtype; o.es = p->dtype == AHAKV_F32 ? 4 : 2;
  o.pool = p->pool_kernel; o.flags = p->flags; o.n_total = p->n_total;
  o.R = G * p->obs_window;
  o.group_max = (p->flags & AHAKV_FLAG_GROUP_MAX) != 0 && G > 1;   // the maximum over one head is that head
  o.n_blk = (o.n + kKeyTile - 1) / kKeyTile;
  if (!resolve_strides(p->q_stride, o.qs, o.Hq, o.r, o.d, o.es) ||
      !resolve_strides(p->k_stride, o.ks, o.Hkv, o.n, o.d, o.es) ||
      !resolve_strides(p->v_stride, o.vs, o.Hkv, o.n, o.d, o.es))
    return AHAKV_ERR_INVALID_ARG;

  for (int i = 0; i < kMaxRows; ++i) { o.rows.c[i] = 0.f; o.lambda[i] = 0.0; o.last[i] = 0; }
  const long long first_cached = p->n_total - p->n_ctx;      // logical position of cache row 0
  for (int i = 0; i < o.r; ++i) {
    const long long pos = obs_pos ? obs_pos[i] : p->n_total - p->obs_window + i;
    if (pos < first_cached || pos >= p->n_total || (i > 0 && obs_pos && pos <= obs_pos[i - 1])) return AHAKV_ERR_INVALID_ARG;
    o.last[i] = (int)(pos - first_cached);
    double lam;
    if (p->scale_mode == AHAKV_SCALE_FIXED) lam = (double)p->scale;
    else if (p->scale_mode == AHAKV_SCALE_ADAPTIVE_ROW) lam = eq12((double)(pos + 1), (double)p->budget, p->head_dim);
    else lam = eq12((double)p->n_total, (double)p->budget, p->head_dim);
    o.lambda[i] = lam;
    o.rows.c[i] = (float)(lam * 1.4426950408889634);
  }

  o.n_eff = o.last[o.r - 1] + 1;

  // Tensor-core scoring: 16-bit inputs.  A row block stacks up to 128 / r query heads of one KV head (one TMA
  // box); when G is not a multiple of that, the last block of each KV head simply holds fewer heads.
  o.heads_per_rb = 1; o.n_rb = 1; o.use_tc = false;
  if (o.es == 2 && o.n >= kKeyTile && (long long)o.B * o.Hkv * 2 * o.n_blk < (1LL << 30) && score_tc_available()) {
    if (o.r <= 128) {
      int hb = 128 / o.r;
      if (hb > G) hb = G;
      if (o.group_max) hb = 1;     // one query head a row block: the blocks' scores are the per-head scores
      o.heads_per_rb = hb;
      o.n_rb = (G + hb - 1) / hb;
      o.use_tc = true;
    } else {              // one query head split over two row blocks
      o.heads_per_rb = 1;
      o.n_rb = 2;
      o.use_tc = (G == 1);
    }
  }
  const int rb_slots = o.use_tc ? o.n_rb : 1;

  const size_t units = (size_t)o.B * o.Hkv;
  size_t off = 0;
  o.off_status = off;  off += 256;
  o.off_sync = off;    off += align_up(units * rb_slots * 2 * sizeof(int), 256);
  o.off_sraw = off;    off += align_up(units * rb_slots * o.n * sizeof(float), 256);
  o.off_nu = off;      off += align_up(units * o.n * sizeof(float), 256);
  o.off_partial = off; off += align_up(units * rb_slots * o.n_blk * (o.use_tc ? 128 : o.R) * sizeof(float2), 256);
  o.off_final = off;   off += align_up(units * rb_slots * (o.use_tc ? 128 : o.R) * sizeof(float2), 256);
  o.off_score = off;   off += align_up(units * o.n * sizeof(float), 256);
  o.ws_total = off;
  return AHAKV_OK;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

static ahakv_status check_ws(const Plan& pl, void* ws, size_t ws_bytes) {
  if (!ws || ((uintptr_t)ws & 255) != 0 || ws_bytes < pl.ws_total) return AHAKV_ERR_WORKSPACE;
  return AHAKV_OK;
}

template <typename T> static T* at(void* ws, size_t off) { return reinterpret_cast<T*>((char*)ws + off); }

// Queues the kernels that leave the raw accumulated score (per row block) and, with the value prior, the value
// norms in the workspace.
static ahakv_status queue_raw_score(const Plan& pl, const void* q, const void* k, const void* v, void* ws,
                                    cudaStream_t st, int prof) {
  TraceRange range("ahakv: score");
  ahakv_status rc = cuda_ok(cudaMemsetAsync(at<char>(ws, pl.off_status), 0, pl.off_sraw - pl.off_status, st));
  if (rc) return rc;
  profile_mark(prof, 0, st);
  float* s_raw = at<float>(ws, pl.off_sraw);
  float2* partial = at<float2>(ws, pl.off_partial);
  float* final_off = at<float>(ws, pl.off_final);
  const bool prior = (pl.flags & AHAKV_FLAG_VALUE_PRIOR) != 0;
  float* nu = prior ? at<float>(ws, pl.off_nu) : nullptr;
  // The tensor-core kernel squares the value rows on its way, as long as its tiles cover all of them: when no
  // observation row sees the last keys it skips their tiles, their raw score is zero and their value rows are
  // squared by the streaming kernel.
  const bool all_keys = pl.n_eff == pl.n;
  const bool tc_prior = prior && pl.use_tc && all_keys;
  if (pl.use_tc && !all_keys &&
      cudaMemsetAsync(s_raw, 0, pl.off_nu - pl.off_sraw, st) != cudaSuccess)
    return AHAKV_ERR_CUDA;
  if (pl.use_tc)
    rc = launch_score_tc(pl, q, k, tc_prior ? v : nullptr, s_raw, nu, partial, at<int>(ws, pl.off_sync),
                         at<int>(ws, pl.off_status), st);
  else
    rc = launch_score_simt(pl, q, k, s_raw, partial, final_off, st);
  if (rc) return rc;
  profile_mark(prof, 1, st);
  if (prior && !tc_prior) {
    rc = launch_vnorm(pl, v, nu, st);
    if (rc) return rc;
  }
  profile_mark(prof, 2, st);
  return AHAKV_OK;
}

static int score_slots(const Plan& pl) { return pl.use_tc ? pl.n_rb : 1; }

}  // namespace ahakv

using namespace ahakv;

extern "C" {

size_t ahakv_workspace_bytes(const ahakv_params* p) {
  Plan pl;
  if (make_plan(p, &pl) != AHAKV_OK) return 0;
  return pl.ws_total;
}

double ahakv_lambda(int64_t n_total, int32_t budget, int32_t head_dim) {
  if (budget < 1 || head_dim < 1) return 0.0;
  return eq12((double)n_total, (double)budget, head_dim);
}

static ahakv_status score_impl(const ahakv_params* p, const int64_t* obs_pos, const void* q_obs, const void* k,
                               const void* v, const float* score_prev, float* score, void* ws, size_t ws_bytes,
                               cudaStream_t st) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl, obs_pos);
  if (rc) return rc;
  const bool prior = (pl.flags & AHAKV_FLAG_VALUE_PRIOR) != 0;
  if (!q_obs || !k || !score || (prior && !v)) return AHAKV_ERR_INVALID_ARG;
  if (!aligned16(q_obs) || !aligned16(k) || (v && !aligned16(v)) || !aligned16(score) ||
      (score_prev && !aligned16(score_prev)))
    return AHAKV_ERR_INVALID_ARG;
  if ((rc = check_ws(pl, ws, ws_bytes))) return rc;
  const int prof = profile_begin_call(st);
  if ((rc = queue_raw_score(pl, q_obs, k, v, ws, st, prof))) return rc;
  rc = launch_refine(pl, at<float>(ws, pl.off_sraw), prior ? at<float>(ws, pl.off_nu) : nullptr, score_prev, score,
                     score_slots(pl), st);
  profile_mark(prof, 3, st);
  profile_mark(prof, 4, st);   // no selection or compaction in this call
  profile_mark(prof, 5, st);
  return rc;
}

ahakv_status ahakv_score(const ahakv_params* p, const void* q_obs, const void* k, const void* v,
                         const float* score_prev, float* score, void* ws, size_t ws_bytes,
                         ahakv_stream_t stream) {
  return score_impl(p, nullptr, q_obs, k, v, score_prev, score, ws, ws_bytes, (cudaStream_t)stream);
}

ahakv_status ahakv_score_rows(const ahakv_params* p, const int64_t* obs_pos, const void* q_obs, const void* k,
                              const void* v, const float* score_prev, float* score, void* ws, size_t ws_bytes,
                              ahakv_stream_t stream) {
  if (!obs_pos) return AHAKV_ERR_INVALID_ARG;
  return score_impl(p, obs_pos, q_obs, k, v, score_prev, score, ws, ws_bytes, (cudaStream_t)stream);
}

ahakv_status ahakv_score_full_causal(const ahakv_params* p, const void* q_all, const void* k, const void* v,
                                     const float* score_prev, float* score, void* ws, size_t ws_bytes,
                                     ahakv_stream_t stream) {
  Plan full;
  ahakv_status rc = make_plan(p, &full);      // validates everything but the query layout; sizes the workspace
  if (rc) return rc;
  if (full.group_max) return AHAKV_ERR_UNSUPPORTED;   // a maximum over heads of sums over passes is not a sum of maxima
  const bool prior = (full.flags & AHAKV_FLAG_VALUE_PRIOR) != 0;
  if (!q_all || !k || !score || (prior && !v)) return AHAKV_ERR_INVALID_ARG;
  if (!aligned16(q_all) || !aligned16(k) || (v && !aligned16(v)) || !aligned16(score) ||
      (score_prev && !aligned16(score_prev)))
    return AHAKV_ERR_INVALID_ARG;
  if ((rc = check_ws(full, ws, ws_bytes))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // q_all holds a query for every cached row: [B, Hq, n, d] unless strides say otherwise
  ahakv_params pc = *p;
  if (p->q_stride[0] == 0 && p->q_stride[1] == 0 && p->q_stride[2] == 0) {
    pc.q_stride[2] = p->head_dim;
    pc.q_stride[1] = (int64_t)p->n_ctx * p->head_dim;
    pc.q_stride[0] = (int64_t)p->n_q_heads * p->n_ctx * p->head_dim;
  }
  pc.flags = p->flags & ~(uint32_t)AHAKV_FLAG_VALUE_PRIOR;     // the prior multiplies the finished sum, once
  float* acc = at<float>(ws, full.off_score);                  // running sum over the passes, [B, Hkv, n]
  const int R = p->obs_window, n = p->n_ctx;
  const long long first_cached = p->n_total - p->n_ctx;
  int64_t pos[kMaxRows];
  for (int c0 = 0; c0 < n; c0 += R) {
    const int rows = n - c0 < R ? n - c0 : R;
    pc.obs_window = rows;
    for (int i = 0; i < rows; ++i) pos[i] = first_cached + c0 + i;
    Plan pl;
    if ((rc = make_plan(&pc, &pl, pos))) return rc;
    if (pl.off_score > full.off_score) return AHAKV_ERR_WORKSPACE;   // cannot happen: fewer rows never need more room
    const char* qc = (const char*)q_all + (size_t)c0 * pl.qs[2] * pl.es;
    if ((rc = queue_raw_score(pl, qc, k, nullptr, ws, st, -1))) return rc;
    if ((rc = launch_refine(pl, at<float>(ws, pl.off_sraw), nullptr, c0 == 0 ? nullptr : acc, acc, score_slots(pl), st)))
      return rc;
  }
  float* nu = nullptr;
  if (prior) {
    nu = at<float>(ws, full.off_nu);
    if ((rc = launch_vnorm(full, v, nu, st))) return rc;
  }
  Plan one = full;
  one.group_max = 0;
  return launch_refine(one, acc, nu, score_prev, score, 1, st);
}

ahakv_status ahakv_score_step(const ahakv_params* p, const void* q_t, const void* k, const float* score_prev,
                              float* score, ahakv_stream_t stream) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl);
  if (rc) return rc;
  if (pl.r != 1) return AHAKV_ERR_INVALID_ARG;
  if (!q_t || !k || !score || !aligned16(q_t) || !aligned16(k) || !aligned16(score) ||
      (score_prev && !aligned16(score_prev)))
    return AHAKV_ERR_INVALID_ARG;
  if ((pl.flags & AHAKV_FLAG_VALUE_PRIOR) || !step_score_fits(pl)) return AHAKV_ERR_UNSUPPORTED;
  return launch_step_score(pl, q_t, k, score_prev, score, (cudaStream_t)stream);
}

ahakv_status ahakv_step_slots(const ahakv_params* p, const void* q_t, const void* k_t, const void* v_t, void* k, void* v,
                              float* score, int32_t* pos, int32_t* free_slot, ahakv_stream_t stream) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl);
  if (rc) return rc;
  if (pl.r != 1 || pl.n != pl.Bud + 1) return AHAKV_ERR_INVALID_ARG;
  if (!q_t || !k_t || !v_t || !k || !v || !score || !pos || !free_slot || !aligned16(q_t) || !aligned16(k_t) ||
      !aligned16(v_t) || !aligned16(k) || !aligned16(v) || ((uintptr_t)score & 3) || ((uintptr_t)pos & 3) ||
      ((uintptr_t)free_slot & 3))
    return AHAKV_ERR_INVALID_ARG;
  if (pl.n_total - 1 > 0x7ffffffe) return AHAKV_ERR_INVALID_ARG;
  if ((pl.flags & AHAKV_FLAG_VALUE_PRIOR) || !step_score_fits(pl)) return AHAKV_ERR_UNSUPPORTED;
  return launch_step_slots(pl, q_t, k_t, v_t, k, v, score, pos, free_slot, (int)(pl.n_total - 1), (cudaStream_t)stream);
}

ahakv_status ahakv_compact_inplace(const ahakv_params* p, void* k, void* v, float* score, const int32_t* kept_idx,
                                   ahakv_stream_t stream) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl);
  if (rc) return rc;
  if (!k || !v || !kept_idx || !aligned16(k) || !aligned16(v) || ((uintptr_t)kept_idx & 3) ||
      (score && ((uintptr_t)score & 3)))
    return AHAKV_ERR_INVALID_ARG;
  return launch_compact_inplace(pl, k, v, score, kept_idx, (cudaStream_t)stream);
}

size_t ahakv_entropy_workspace_bytes(const ahakv_params* p) {
  Plan pl;
  if (make_plan(p, &pl) != AHAKV_OK) return 0;
  return entropy_scratch_bytes(pl);
}

ahakv_status ahakv_row_entropy(const ahakv_params* p, const void* q_obs, const void* k, float* entropy, void* ws,
                               size_t ws_bytes, ahakv_stream_t stream) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl);
  if (rc) return rc;
  if (!q_obs || !k || !entropy || !aligned16(q_obs) || !aligned16(k) || ((uintptr_t)entropy & 3))
    return AHAKV_ERR_INVALID_ARG;
  if (!ws || ((uintptr_t)ws & 255) != 0 || ws_bytes < entropy_scratch_bytes(pl)) return AHAKV_ERR_WORKSPACE;
  return launch_entropy(pl, q_obs, k, ws, entropy, (cudaStream_t)stream);
}

ahakv_status ahakv_select(const ahakv_params* p, const float* score, int32_t* kept_idx, void* ws,
                          size_t ws_bytes, ahakv_stream_t stream) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl);
  if (rc) return rc;
  if (!score || !kept_idx || !aligned16(score) || ((uintptr_t)kept_idx & 3)) return AHAKV_ERR_INVALID_ARG;
  (void)ws; (void)ws_bytes;                    // selection works in shared memory: no scratch is needed
  return launch_select(pl, score, kept_idx, nullptr, (cudaStream_t)stream);
}

ahakv_status ahakv_compact(const ahakv_params* p, const void* k, const void* v, const float* score,
                           const int32_t* kept_idx, void* k_out, void* v_out, float* score_out,
                           ahakv_stream_t stream) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl);
  if (rc) return rc;
  if (!k || !v || !kept_idx || !k_out || !v_out) return AHAKV_ERR_INVALID_ARG;
  if ((score == nullptr) != (score_out == nullptr)) return AHAKV_ERR_INVALID_ARG;
  if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out) || ((uintptr_t)kept_idx & 3))
    return AHAKV_ERR_INVALID_ARG;
  return launch_compact(pl, k, v, score, kept_idx, k_out, v_out, score_out, (cudaStream_t)stream);
}

static ahakv_status evict_impl(const ahakv_params* p, const int32_t* budgets, const void* q_obs, const void* k,
                               const void* v, const float* score_prev, void* k_out, void* v_out, float* score_out,
                               int32_t* kept_idx, void* ws, size_t ws_bytes, ahakv_stream_t stream) {
  Plan pl;
  ahakv_status rc = make_plan(p, &pl);
  if (rc) return rc;
  if (!q_obs || !k || !v || !k_out || !v_out || !kept_idx) return AHAKV_ERR_INVALID_ARG;
  if (!aligned16(q_obs) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out) ||
      ((uintptr_t)kept_idx & 3) || (score_prev && !aligned16(score_prev)))
    return AHAKV_ERR_INVALID_ARG;
  if ((rc = check_ws(pl, ws, ws_bytes))) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  TraceRange call("ahakv_evict");
  const int prof = profile_begin_call(st);
  if ((rc = queue_raw_score(pl, q_obs, k, v, ws, st, prof))) return rc;
  const bool prior = (pl.flags & AHAKV_FLAG_VALUE_PRIOR) != 0;
  float* s_raw = at<float>(ws, pl.off_sraw);
  float* nu = prior ? at<float>(ws, pl.off_nu) : nullptr;
  float* score = at<float>(ws, pl.off_score);
  nvtxRangePushA("ahakv: refine + select");
  if (refine_select_fits(pl)) {      // a head's scores fit in one CTA's registers: both steps in one launch
    rc = launch_refine_select(pl, s_raw, nu, score_prev, score, kept_idx, score_slots(pl), budgets, st);
    profile_mark(prof, 3, st);
  } else {
    rc = launch_refine(pl, s_raw, nu, score_prev, score, score_slots(pl), st);
    profile_mark(prof, 3, st);
    if (rc == AHAKV_OK) rc = launch_select(pl, score, kept_idx, budgets, st);
  }
  nvtxRangePop();
  profile_mark(prof, 4, st);
  {
    TraceRange range("ahakv: compact");
    if (rc == AHAKV_OK) rc = launch_compact(pl, k, v, score_out ? score : nullptr, kept_idx, k_out, v_out, score_out, st);
  }
  profile_mark(prof, 5, st);
  return rc;
}

ahakv_status ahakv_evict(const ahakv_params* p, const void* q_obs, const void* k, const void* v,
                         const float* score_prev, void* k_out, void* v_out, float* score_out,
                         int32_t* kept_idx, void* ws, size_t ws_bytes, ahakv_stream_t stream) {
  return evict_impl(p, nullptr, q_obs, k, v, score_prev, k_out, v_out, score_out, kept_idx, ws, ws_bytes, stream);
}

ahakv_status ahakv_evict_head_budgets(const ahakv_params* p, const int32_t* head_budget, const void* q_obs, const void* k,
                                      const void* v, const float* score_prev, void* k_out, void* v_out,
                                      float* score_out, int32_t* kept_idx, void* ws, size_t ws_bytes,
                                      ahakv_stream_t stream) {
  if (!head_budget || ((uintptr_t)head_budget & 3)) return AHAKV_ERR_INVALID_ARG;
  return evict_impl(p, head_budget, q_obs, k, v, score_prev, k_out, v_out, score_out, kept_idx, ws, ws_bytes, stream);
}

ahakv_status ahakv_evict_ragged(const ahakv_params* p, const ahakv_seq* seqs, const void* q_obs, const void* k,
                                const void* v, const float* score_prev, void* k_out, void* v_out, float* score_out,
                                int32_t* kept_idx, void* ws, size_t ws_bytes, ahakv_stream_t stream) {
  Plan outer;
  ahakv_status rc = make_plan(p, &outer);        // p describes the allocation: n_ctx and budget are the largest of the batch
  if (rc) return rc;
  if (!seqs) return AHAKV_ERR_INVALID_ARG;
  if ((rc = check_ws(outer, ws, ws_bytes))) return rc;
  // every sequence is checked before anything is queued
  for (int b = 0; b < outer.B; ++b) {
    if (seqs[b].n_ctx < outer.r || seqs[b].n_ctx > p->n_ctx || seqs[b].budget < 1 || seqs[b].budget > p->budget ||
        seqs[b].budget < p->recent_window || seqs[b].n_total < seqs[b].n_ctx)
      return AHAKV_ERR_INVALID_ARG;
  }
  const size_t es = outer.es, keep_max = outer.n_keep;
  const size_t row = (size_t)outer.d * es;
  for (int b = 0; b < outer.B; ++b) {
    ahakv_params pb = *p;
    pb.batch = 1;
    pb.n_ctx = seqs[b].n_ctx;
    pb.n_total = seqs[b].n_total;
    pb.budget = seqs[b].budget;
    for (int t = 0; t < 3; ++t) { pb.q_stride[t] = outer.qs[t]; pb.k_stride[t] = outer.ks[t]; pb.v_stride[t] = outer.vs[t]; }
    const char* qb = (const char*)q_obs + (size_t)b * outer.qs[0] * es;
    const char* kb = (const char*)k + (size_t)b * outer.ks[0] * es;
    const char* vb = (const char*)v + (size_t)b * outer.vs[0] * es;
    const size_t tok = (size_t)b * outer.Hkv * outer.n, kept = (size_t)b * outer.Hkv * keep_max;
    rc = ahakv_evict(&pb, qb, kb, vb, score_prev ? score_prev + tok : nullptr, (char*)k_out + kept * row,
                     (char*)v_out + kept * row, score_out ? score_out + kept : nullptr, kept_idx + kept, ws, ws_bytes,
                     stream);
    if (rc) return rc;
  }
  return AHAKV_OK;
}

ahakv_status ahakv_last_device_status(const void* ws, ahakv_stream_t stream) {
  if (!ws) return AHAKV_ERR_WORKSPACE;
  int word = 0;
  if (cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
    return AHAKV_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return AHAKV_ERR_CUDA;
  return word == 0 ? AHAKV_OK : AHAKV_ERR_TIMEOUT;
}

void ahakv_test_set_wait(int32_t wait_ms, int32_t withhold_first_partial) {
  score_tc_test_hooks((long long)wait_ms * 1000000LL, withhold_first_partial != 0);
}

int64_t ahakv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* ahakv_status_string(ahakv_status s) {
  switch (s) {
    case AHAKV_OK: return "ok";
    case AHAKV_ERR_INVALID_ARG: return "invalid argument";
    case AHAKV_ERR_UNSUPPORTED: return "unsupported request";
    case AHAKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case AHAKV_ERR_CUDA: return "CUDA call or launch failed";
    case AHAKV_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

}  // extern "C"
