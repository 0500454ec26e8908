// Host side of the C ABI: argument validation, work-space layout and the launch sequences.
#include <algorithm>
#include <atomic>
#include <string>
#include <cstring>
#include <mutex>

#include "ckv_common.cuh"

namespace ckv {

static std::atomic<int64_t> g_launches{0};
static std::atomic<int> g_score_path{0};  // 0 = automatic, 1 = plain kernels, 2 = tensor-core kernel
static std::atomic<int> g_pdl{1};         // 1: the kernels after the pooling kernel use programmatic dependent launch
static std::atomic<int> g_group_fuse{1};  // 1: the scan writes per-group maxima and masses where it can
static std::atomic<int> g_run_tiles{16};  // key tiles per run of the tensor-core scan
static std::atomic<int> g_l2_hints{1};    // 1: first-pass K loads keep their lines in L2, second-pass loads release them
static std::atomic<unsigned long long> g_wait_limit_ns{2000000000ull};   // bound of every device-side wait
unsigned long long wait_limit_ns() { return g_wait_limit_ns.load(std::memory_order_relaxed); }
static thread_local cudaEvent_t t_scan_start = nullptr, t_scan_stop = nullptr;  // see ckv_set_scan_events

// The scheduling settings of one call: params->tuning where it gives a value, the process-wide defaults elsewhere.
// An entry point resolves them once and makes them current for its thread while it queues its launches, so that the
// launchers need no extra arguments and concurrent calls on other threads keep their own.
struct CallTuning {
  int score_path, run_tiles, l2_hints, group_fuse, pdl;
  cudaEvent_t ev0, ev1;
};
static thread_local const CallTuning* t_call = nullptr;
static CallTuning resolve_tuning(const ckv_params& p) {
  const ckv_tuning* t = p.tuning;
  CallTuning c;
  c.score_path = t && t->score_path >= 0 ? t->score_path : g_score_path.load(std::memory_order_relaxed);
  c.run_tiles = t && t->run_tiles >= 0 ? t->run_tiles : g_run_tiles.load(std::memory_order_relaxed);
  c.l2_hints = t && t->l2_hints >= 0 ? t->l2_hints : g_l2_hints.load(std::memory_order_relaxed);
  c.group_fuse = t && t->group_fuse >= 0 ? t->group_fuse : g_group_fuse.load(std::memory_order_relaxed);
  c.pdl = t && t->pdl >= 0 ? t->pdl : g_pdl.load(std::memory_order_relaxed);
  c.ev0 = t && t->scan_start_event ? (cudaEvent_t)t->scan_start_event : t_scan_start;
  c.ev1 = t && t->scan_stop_event ? (cudaEvent_t)t->scan_stop_event : t_scan_stop;
  return c;
}
struct TuningScope {
  CallTuning mine;
  const CallTuning* outer;
  explicit TuningScope(const ckv_params& p) : mine(resolve_tuning(p)), outer(t_call) { t_call = &mine; }
  ~TuningScope() { t_call = outer; }
};
bool pdl_enabled() { return (t_call ? t_call->pdl : g_pdl.load(std::memory_order_relaxed)) != 0; }
int tuning_run_tiles() { return t_call ? t_call->run_tiles : g_run_tiles.load(std::memory_order_relaxed); }
int tuning_l2_hints() { return t_call ? t_call->l2_hints : g_l2_hints.load(std::memory_order_relaxed); }
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }
static ckv_status noalloc_scratch(char** out);   // device address of the fixed scratch (end of this file)

WsLayout ws_layout(const ckv_shape& s, const ckv_params& p) {
  WsLayout w{};
  const size_t Nu = s.n_units, H = s.n_q_heads, Hkv = s.n_kv_heads, L = s.seq_len, W = s.window;
  const size_t n = L - W;
  w.nblk = (int)((L + kPlainKeysPerBlock - 1) / kPlainKeysPerBlock);
  size_t o = 0;
  // what the score stage touches comes first, so that its extent alone decides whether a problem fits a small
  // fixed scratch (ckv_score_noalloc)
  w.status = o, o += 256;
  if (s.dtype == CKV_BF16) w.tc_flags = o, o = align_up(o + tc_layout(s).flag_bytes);   // behind the status words: one kernel clears both
  w.csum = o, o = align_up(o + Nu * H * L * sizeof(float));
  w.part = o, o = align_up(o + Nu * H * W * (size_t)w.nblk * sizeof(float2));
  w.stat = o, o = align_up(o + Nu * H * W * sizeof(float2));
  {
    const BudgetLayout b = budget_layout(s);
    w.ent_part = o, o = align_up(o + b.ent_bytes);
    w.bud_done = o, o = align_up(o + b.done_bytes);
    if (s.dtype == CKV_BF16) {
      const TcLayout t = tc_layout(s);
      w.tc_part = o, o = align_up(o + t.part_bytes);
      w.tc_stat = o, o = align_up(o + t.stat_bytes);
    }
    w.score_extent = o;
    w.cnt_part = o, o = align_up(o + b.cnt_bytes);
  }
  w.colmass = o, o = align_up(o + Nu * L * sizeof(float));
  w.scores = o, o = align_up(o + Nu * Hkv * (n ? n : 1) * sizeof(float));
  w.bucket = o, o = align_up(o + Nu * sizeof(int32_t));
  w.entropy = o, o = align_up(o + Nu * sizeof(float));
  w.pmass = o, o = align_up(o + (p.global_alpha ? Nu / (size_t)p.units_per_prompt * L * sizeof(float) : 0));
  {
    const size_t slots = Nu * Hkv * (size_t)attend_slices(s) * kAttendMaxRows;
    w.att_ml = o, o = align_up(o + slots * sizeof(float2));
    w.att_o = o, o = align_up(o + slots * kHeadDim * sizeof(float));
  }
  w.vn_part = o, o = align_up(o + Nu * Hkv * ((L + kVnormRows - 1) / kVnormRows) * sizeof(float));
  w.vn_rho = o, o = align_up(o + (p.value_norm ? Nu * Hkv * L * sizeof(float) : 0));
  w.total = o;
  return w;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static ckv_status check_shape(const ckv_shape* s) {
  if (!s) return CKV_ERR_INVALID_ARG;
  if (s->n_units < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->seq_len < 1 || s->window < 1)
    return CKV_ERR_INVALID_ARG;
  if (s->n_q_heads % s->n_kv_heads) return CKV_ERR_INVALID_ARG;
  if (s->window > s->seq_len) return CKV_ERR_INVALID_ARG;
  if (s->dtype != CKV_BF16 && s->dtype != CKV_F32) return CKV_ERR_INVALID_ARG;
  if (s->head_dim != kHeadDim || s->window > kMaxWindow || s->n_kv_heads > kMaxKvHeads) return CKV_ERR_UNSUPPORTED;
  if (s->n_units > 65535 || s->n_q_heads > 65535) return CKV_ERR_UNSUPPORTED;
  if (s->seq_len > (1 << 20)) return CKV_ERR_UNSUPPORTED;
  const int64_t esz = s->dtype == CKV_BF16 ? 2 : 4;
  const int64_t strides[6] = {s->q_stride_unit, s->q_stride_head,  s->q_stride_row,
                              s->kv_stride_unit, s->kv_stride_head, s->kv_stride_tok};
  for (int64_t st : strides)
    if (st < 0 || (st * esz) % 16) return CKV_ERR_INVALID_ARG;
  if (s->q_stride_row < kHeadDim || s->kv_stride_tok < kHeadDim) return CKV_ERR_INVALID_ARG;
  // a zero stride over more than one element (a broadcast view) is refused: the tensor maps of the scan cannot
  // describe it, and no caller of a retention pass has two units or heads that share their rows
  if ((s->n_units > 1 && (s->q_stride_unit == 0 || s->kv_stride_unit == 0)) ||
      (s->n_q_heads > 1 && s->q_stride_head == 0) || (s->n_kv_heads > 1 && s->kv_stride_head == 0))
    return CKV_ERR_INVALID_ARG;
  return CKV_OK;
}

static ckv_status check_params(const ckv_shape* s, const ckv_params* p) {
  if (!p) return CKV_ERR_INVALID_ARG;
  if (p->pool_kind < CKV_POOL_NONE || p->pool_kind > CKV_POOL_AVG) return CKV_ERR_INVALID_ARG;
  if (p->pool_size < 1 || p->pool_size > 15 || (p->pool_size & 1) == 0) return CKV_ERR_INVALID_ARG;
  if (p->budget_per_head < 1 || p->floor_per_head < 0 || p->n_buckets < 1) return CKV_ERR_INVALID_ARG;
  if (p->bucket_override < -1 || p->bucket_override >= p->n_buckets) return CKV_ERR_INVALID_ARG;
  if (p->head_w_stride_unit < 0 || p->sens_stride_unit < 0) return CKV_ERR_INVALID_ARG;
  if (p->value_norm != 0 && p->value_norm != 1) return CKV_ERR_INVALID_ARG;
  if (const ckv_tuning* t = p->tuning) {
    if (t->score_path < -1 || t->score_path > 2 || t->run_tiles < -1 || t->run_tiles == 0 || t->run_tiles > 64 ||
        t->l2_hints < -1 || t->l2_hints > 1 || t->group_fuse < -1 || t->group_fuse > 1 || t->pdl < -1 || t->pdl > 1)
      return CKV_ERR_INVALID_ARG;
  }
  if (p->shared_elastic != 0 && p->shared_elastic != 1) return CKV_ERR_INVALID_ARG;
  if (p->global_alpha != 0 && p->global_alpha != 1) return CKV_ERR_INVALID_ARG;
  if (p->units_per_prompt < 0) return CKV_ERR_INVALID_ARG;
  if (p->global_alpha && (p->units_per_prompt < 1 || s->n_units % p->units_per_prompt)) return CKV_ERR_INVALID_ARG;
  if (!(p->value_norm_eps >= 0.f) || !(p->value_norm_eps < 3.0e38f)) return CKV_ERR_INVALID_ARG;
  if (p->n_gate_layers < 0 || p->n_ppl_bins < 0 || p->n_budget_levels < 0) return CKV_ERR_INVALID_ARG;
  if (p->gate_coords) {   // the four-axis gate table: one dense table for all units
    if (p->n_gate_layers < 1 || p->n_ppl_bins < 1 || p->n_budget_levels < 1 || p->sens_stride_unit != 0)
      return CKV_ERR_INVALID_ARG;
    if (!aligned(p->gate_coords, 4)) return CKV_ERR_INVALID_ARG;
    if ((int64_t)p->n_gate_layers * p->n_buckets * p->n_ppl_bins * p->n_budget_levels > (int64_t)1 << 30)
      return CKV_ERR_UNSUPPORTED;
  }
  if (p->budget_per_head < s->seq_len) {
    if (p->budget_per_head < s->window) return CKV_ERR_INVALID_ARG;
    if (p->floor_per_head > p->budget_per_head - s->window) return CKV_ERR_INVALID_ARG;
  }
  return CKV_OK;
}

static ckv_status check_ws(const ckv_shape* s, const ckv_params* p, const void* ws, size_t ws_bytes) {
  if (!ws || !aligned(ws, 256) || ws_bytes < ws_layout(*s, *p).total) return CKV_ERR_WORKSPACE;
  return CKV_OK;
}

static bool all_aligned16(std::initializer_list<const void*> ps) {
  for (const void* p : ps)
    if (!p || !aligned(p, 16)) return false;
  return true;
}
static bool all_aligned4(std::initializer_list<const void*> ps) {
  for (const void* p : ps)
    if (!p || !aligned(p, 4)) return false;
  return true;
}

#define CKV_TRY(expr)                  \
  do {                                 \
    ckv_status st__ = (expr);          \
    if (st__ != CKV_OK) return st__;   \
  } while (0)
#define CKV_CUDA(expr)                               \
  do {                                               \
    if ((expr) != cudaSuccess) return CKV_ERR_CUDA;  \
  } while (0)

// Word kStatusMagicWord of the status section says that words 0..7 (the status code and the waits that were in
// progress when it was set) are meaningful; a work space seen for the first time has them cleared.  The words
// behind them (counters, the scan's flags and queues) are cleared on every call.
constexpr int kStatusMagicWord = 63;
constexpr int kStatusMagic = 0x434b5631;
__global__ void ws_reset_kernel(int* status, size_t n_flag_words) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x, step = (size_t)gridDim.x * blockDim.x;
  if (i == 0 && status[kStatusMagicWord] != kStatusMagic) {
    for (int w = 0; w < 8; ++w) status[w] = 0;
    status[kStatusMagicWord] = kStatusMagic;
  }
  if (i >= 8 && i < (size_t)kStatusMagicWord) status[i] = 0;
  int* flags = status + 64;
  for (size_t w = i; w < n_flag_words; w += step) flags[w] = 0;
}
static cudaError_t launch_ws_reset(int* status, size_t n_flag_words, cudaStream_t st) {
  const int blocks = (int)std::min<size_t>(64, (n_flag_words + 255) / 256 + 1);
  ws_reset_kernel<<<blocks, 256, 0, st>>>(status, n_flag_words);
  count_launch();
  return cudaGetLastError();
}

static ckv_status score_impl(const ckv_shape& s, const ckv_params& p, const void* q, const void* k,
                             const float* head_w, float* scores, float* colmass, char* ws, cudaStream_t st) {
  const WsLayout w = ws_layout(s, p);
  const CallTuning tune = t_call ? *t_call : resolve_tuning(p);
  const int path = tune.score_path;
  const bool tc_ok = score_tc_supported(s) && s.seq_len >= 128;
  if (path == 2 && !tc_ok) return CKV_ERR_UNSUPPORTED;
  const bool use_tc = tc_ok && path != 1;
  // the scheduler words and, behind them, the tensor-core scan's counters and run queues start at zero; the
  // status words keep a code that no ckv_device_status call has read yet
  CKV_CUDA(launch_ws_reset(reinterpret_cast<int*>(ws + w.status), use_tc ? tc_layout(s).flag_bytes / sizeof(int) : 0, st));
  float* csum = reinterpret_cast<float*>(ws + w.csum);
  const cudaEvent_t ev0 = tune.ev0, ev1 = tune.ev1;
  int* marker = reinterpret_cast<int*>(ws + w.status) + kPathMarkerWord;   // who wrote the row statistics
  if (use_tc) {
    // grouped output where it applies: both arrays fit the per-head region (at least two heads per group)
    TcGrouped grp{csum, csum + (int64_t)s.n_units * s.n_kv_heads * s.seq_len, head_w, p.head_w_stride_unit};
    const bool grouped = score_tc_groupable(s, p) && tune.group_fuse != 0;
    if (ev0) CKV_CUDA(cudaEventRecord(ev0, st));
    CKV_CUDA(launch_score_tc(s, q, k, csum, grouped ? &grp : nullptr, ws + w.tc_part, ws + w.tc_stat,
                             reinterpret_cast<int*>(ws + w.tc_flags), reinterpret_cast<int*>(ws + w.status), st));
    if (ev1) CKV_CUDA(cudaEventRecord(ev1, st));
    if (grouped) {
      CKV_CUDA(launch_epilogue_grouped(s, p, grp.zgrp, grp.mgrp, scores, colmass, ws + w.ent_part, ws + w.bud_done,
                                       marker, 2, st));
      return CKV_OK;
    }
  } else {
    CKV_CUDA(launch_score_plain(s, q, k, csum, reinterpret_cast<float2*>(ws + w.part),
                                reinterpret_cast<float2*>(ws + w.stat), w.nblk, st));
  }
  CKV_CUDA(launch_epilogue(s, p, csum, head_w, scores, colmass, ws + w.ent_part, ws + w.bud_done, marker,
                           use_tc ? 2 : 1, st));
  return CKV_OK;
}

}  // namespace ckv

using namespace ckv;

#pragma GCC visibility push(default)
extern "C" {

size_t ckv_workspace_bytes(const ckv_shape* shape, const ckv_params* params) {
  if (check_shape(shape) != CKV_OK || check_params(shape, params) != CKV_OK) return 0;
  return ws_layout(*shape, *params).total;
}

size_t ckv_score_workspace_bytes(const ckv_shape* shape, const ckv_params* params) {
  if (check_shape(shape) != CKV_OK || check_params(shape, params) != CKV_OK) return 0;
  return ws_layout(*shape, *params).score_extent;
}

ckv_status ckv_score(const ckv_shape* shape, const ckv_params* params, const void* q_win, const void* k,
                     const float* head_w, float* scores, float* colmass, void* ws, size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned16({q_win, k}) || !all_aligned4({head_w, scores, colmass})) return CKV_ERR_INVALID_ARG;
  // the score stage alone uses the leading sections of the work space
  if (!ws || !aligned(ws, 256) || ws_bytes < ws_layout(*shape, *params).score_extent) return CKV_ERR_WORKSPACE;
  return score_impl(*shape, *params, q_win, k, head_w, scores, colmass, (char*)ws, (cudaStream_t)stream);
}

ckv_status ckv_budget(const ckv_shape* shape, const ckv_params* params, const float* scores, const float* colmass,
                      const float* sens, int32_t* budgets, int32_t* offsets, int32_t* bucket, float* entropy,
                      void* ws, size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned4({scores, colmass, sens, budgets, offsets, bucket, entropy})) return CKV_ERR_INVALID_ARG;
  CKV_TRY(check_ws(shape, params, ws, ws_bytes));
  const WsLayout w = ws_layout(*shape, *params);
  char* base = (char*)ws;
  CKV_CUDA(launch_entropy_partials(*shape, colmass, base + w.ent_part, base + w.bud_done, (cudaStream_t)stream));
  CKV_CUDA(launch_budget(*shape, *params, scores, sens, budgets, offsets, bucket, entropy, base + w.ent_part,
                         base + w.cnt_part, base + w.bud_done, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_vnorm(const ckv_shape* shape, const ckv_params* params, const void* v, float* rho,
                     float* scores_or_null, void* ws, size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned16({v}) || !all_aligned4({rho})) return CKV_ERR_INVALID_ARG;
  if (scores_or_null && !aligned(scores_or_null, 4)) return CKV_ERR_INVALID_ARG;
  CKV_TRY(check_ws(shape, params, ws, ws_bytes));
  const WsLayout w = ws_layout(*shape, *params);
  float* part = reinterpret_cast<float*>((char*)ws + w.vn_part);
  CKV_CUDA(launch_vnorm_rows(*shape, v, rho, part, (cudaStream_t)stream));
  CKV_CUDA(launch_vnorm_finish(*shape, params->value_norm_eps, rho, part, scores_or_null, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_attend(const ckv_shape* shape, const ckv_params* params, const void* q_dec, int32_t n_dec,
                      const void* k, const void* v, int32_t compressed, const int32_t* budgets, const int32_t* offsets,
                      float* out, float* lse, void* ws, size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (n_dec < 1 || (shape->n_q_heads / shape->n_kv_heads) * n_dec > kAttendMaxRows) return CKV_ERR_UNSUPPORTED;
  if (compressed != 0 && compressed != 1) return CKV_ERR_INVALID_ARG;
  if (!all_aligned16({q_dec, k, v}) || !all_aligned4({out, lse})) return CKV_ERR_INVALID_ARG;
  if (compressed && !all_aligned4({budgets, offsets})) return CKV_ERR_INVALID_ARG;
  CKV_TRY(check_ws(shape, params, ws, ws_bytes));
  const WsLayout w = ws_layout(*shape, *params);
  char* base = (char*)ws;
  CKV_CUDA(launch_attend(*shape, *params, q_dec, n_dec, k, v, compressed, budgets, offsets, out, lse, base + w.att_ml,
                         base + w.att_o, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_kept_mass(const ckv_shape* shape, const ckv_params* params, const void* q_win, const void* k_out,
                         const int32_t* indices, const int32_t* budgets, const int32_t* offsets, float* kept, void* ws,
                         size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned16({q_win, k_out}) || !all_aligned4({indices, budgets, offsets, kept})) return CKV_ERR_INVALID_ARG;
  CKV_TRY(check_ws(shape, params, ws, ws_bytes));
  const WsLayout w = ws_layout(*shape, *params);
  char* base = (char*)ws;
  CKV_CUDA(launch_kept_mass(*shape, *params, q_win, k_out, indices, budgets, offsets, base + w.stat, base + w.tc_stat,
                            reinterpret_cast<const int*>(base + w.status) + kPathMarkerWord, kept,
                            (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_prompt_mass(const ckv_shape* shape, const ckv_params* params, const float* colmass, float* pmass,
                           void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!params->global_alpha || !all_aligned4({colmass, pmass})) return CKV_ERR_INVALID_ARG;
  CKV_CUDA(launch_prompt_mass(*shape, *params, colmass, pmass, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_global_scores(const ckv_shape* shape, const ckv_params* params, const float* head_w,
                             const float* pmass, int32_t units_total, float* scores, float* colmass, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!params->global_alpha || units_total < params->units_per_prompt) return CKV_ERR_INVALID_ARG;
  if (!all_aligned4({head_w, pmass, scores, colmass})) return CKV_ERR_INVALID_ARG;
  CKV_CUDA(launch_global_scores(*shape, *params, units_total, head_w, pmass, scores, colmass, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_unit_max(const ckv_shape* shape, const ckv_params* params, float* scores, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned4({scores})) return CKV_ERR_INVALID_ARG;
  CKV_CUDA(launch_unit_max(*shape, scores, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_select(const ckv_shape* shape, const ckv_params* params, const float* scores, const int32_t* budgets,
                      const int32_t* offsets, int32_t* indices, void* ws, size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned4({scores, budgets, offsets, indices})) return CKV_ERR_INVALID_ARG;
  CKV_TRY(check_ws(shape, params, ws, ws_bytes));
  int* status = reinterpret_cast<int*>(static_cast<char*>(ws) + ws_layout(*shape, *params).status);
  CKV_CUDA(launch_select(*shape, *params, scores, budgets, offsets, indices, status, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_gather(const ckv_shape* shape, const ckv_params* params, const void* k, const void* v,
                      const int32_t* indices, const int32_t* offsets, void* k_out, void* v_out, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned16({k, v, k_out, v_out}) || !all_aligned4({indices, offsets})) return CKV_ERR_INVALID_ARG;
  CKV_CUDA(launch_gather(*shape, *params, k, v, indices, offsets, k_out, v_out, (cudaStream_t)stream));
  return CKV_OK;
}

ckv_status ckv_compress(const ckv_shape* shape, const ckv_params* params, const void* q_win, const void* k,
                        const void* v, const float* head_w, const float* sens, void* k_out, void* v_out,
                        int32_t* indices, int32_t* budgets, int32_t* offsets, float* scores_or_null,
                        int32_t* bucket_or_null, float* entropy_or_null, void* ws, size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned16({q_win, k, v, k_out, v_out}) || !all_aligned4({head_w, sens, indices, budgets, offsets}))
    return CKV_ERR_INVALID_ARG;
  if ((scores_or_null && !aligned(scores_or_null, 4)) || (bucket_or_null && !aligned(bucket_or_null, 4)) ||
      (entropy_or_null && !aligned(entropy_or_null, 4)))
    return CKV_ERR_INVALID_ARG;
  CKV_TRY(check_ws(shape, params, ws, ws_bytes));
  const WsLayout w = ws_layout(*shape, *params);
  char* base = (char*)ws;
  cudaStream_t st = (cudaStream_t)stream;
  float* scores = scores_or_null ? scores_or_null : reinterpret_cast<float*>(base + w.scores);
  float* colmass = reinterpret_cast<float*>(base + w.colmass);
  int32_t* bucket = bucket_or_null ? bucket_or_null : reinterpret_cast<int32_t*>(base + w.bucket);
  float* entropy = entropy_or_null ? entropy_or_null : reinterpret_cast<float*>(base + w.entropy);
  CKV_TRY(score_impl(*shape, *params, q_win, k, head_w, scores, colmass, base, st));
  if (params->global_alpha) {   // Alg. 1 (A): one alpha per prompt, all of whose units are in this call
    float* pmass = reinterpret_cast<float*>(base + w.pmass);
    CKV_CUDA(launch_prompt_mass(*shape, *params, colmass, pmass, st));
    CKV_CUDA(launch_global_scores(*shape, *params, params->units_per_prompt, head_w, pmass, scores, colmass, st));
    // the pooling kernel left entropy partials of the per-unit mass: redo them for the prompt's
    CKV_CUDA(launch_entropy_partials(*shape, colmass, base + w.ent_part, base + w.bud_done, st));
  }
  if (params->value_norm) {   // Eq. 4: u = alpha * rho, before the thresholds see the scores
    float* rho = reinterpret_cast<float*>(base + w.vn_rho);
    float* part = reinterpret_cast<float*>(base + w.vn_part);
    CKV_CUDA(launch_vnorm_rows(*shape, v, rho, part, st));
    CKV_CUDA(launch_vnorm_finish(*shape, params->value_norm_eps, rho, part, scores, st));
  }
  if (params->shared_elastic) CKV_CUDA(launch_unit_max(*shape, scores, st));
  CKV_CUDA(launch_budget(*shape, *params, scores, sens, budgets, offsets, bucket, entropy, base + w.ent_part,
                         base + w.cnt_part, base + w.bud_done, st));
  CKV_CUDA(launch_select(*shape, *params, scores, budgets, offsets, indices, reinterpret_cast<int*>(base + w.status), st));
  CKV_CUDA(launch_gather(*shape, *params, k, v, indices, offsets, k_out, v_out, st));
  return CKV_OK;
}

// Device address under which a kernel can read a host buffer in place (page-locked memory that the device has
// mapped), or null when the buffer has to be copied.
static const void* mapped_host_pointer(const void* host) {
  cudaPointerAttributes at{};
  if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
    (void)cudaGetLastError();
    return nullptr;
  }
  return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

int ckv_reads_in_place(const void* host_pointer) { return host_pointer && mapped_host_pointer(host_pointer) ? 1 : 0; }

// staging sections: q | k | v | head_w | sens | k_out | v_out | indices | budgets | offsets
struct Staging {
  size_t q, k, v, head_w, sens, k_out, v_out, indices, budgets, offsets, total;
  size_t q_b, kv_b, hw_b, sens_b, out_b, idx_b, bud_b, off_b;
  size_t coords, coords_b;   // gate coordinates [Nu,3] (only with the four-axis gate table)
};
static Staging staging_layout(const ckv_shape& s, const ckv_params& p) {
  Staging g{};
  const size_t esz = s.dtype == CKV_BF16 ? 2 : 4;
  const size_t Nu = s.n_units, H = s.n_q_heads, Hkv = s.n_kv_heads, L = s.seq_len, W = s.window, d = s.head_dim;
  const size_t rows = Hkv * (size_t)(p.budget_per_head < s.seq_len ? p.budget_per_head : s.seq_len);
  g.q_b = Nu * H * W * d * esz;
  g.kv_b = Nu * Hkv * L * d * esz;
  g.hw_b = (p.head_w_stride_unit ? Nu : 1) * H * sizeof(float);
  g.sens_b = (p.sens_stride_unit ? Nu : 1) * (size_t)p.n_buckets * sizeof(float);
  if (p.gate_coords) g.sens_b = (size_t)p.n_gate_layers * p.n_buckets * p.n_ppl_bins * p.n_budget_levels * sizeof(float);
  g.coords_b = p.gate_coords ? Nu * 3 * sizeof(int32_t) : 0;
  g.out_b = Nu * rows * d * esz;
  g.idx_b = Nu * rows * sizeof(int32_t);
  g.bud_b = Nu * Hkv * sizeof(int32_t);
  g.off_b = Nu * (Hkv + 1) * sizeof(int32_t);
  size_t o = 0;
  g.q = o, o = align_up(o + g.q_b);
  g.k = o, o = align_up(o + g.kv_b);
  g.v = o, o = align_up(o + g.kv_b);
  g.head_w = o, o = align_up(o + g.hw_b);
  g.sens = o, o = align_up(o + g.sens_b);
  g.k_out = o, o = align_up(o + g.out_b);
  g.v_out = o, o = align_up(o + g.out_b);
  g.indices = o, o = align_up(o + g.idx_b);
  g.budgets = o, o = align_up(o + g.bud_b);
  g.offsets = o, o = align_up(o + g.off_b);
  g.coords = o, o = align_up(o + g.coords_b);
  g.total = o;
  return g;
}

size_t ckv_staging_bytes(const ckv_shape* shape, const ckv_params* params) {
  if (check_shape(shape) != CKV_OK || check_params(shape, params) != CKV_OK) return 0;
  return staging_layout(*shape, *params).total;
}

ckv_status ckv_compress_host(const ckv_shape* shape, const ckv_params* params, const void* q_win_host,
                             const void* k_host, const void* v_host, const float* head_w_host,
                             const float* sens_host, void* k_out_host, void* v_out_host, int32_t* indices_host,
                             int32_t* budgets_host, int32_t* offsets_host, void* staging, size_t staging_bytes,
                             void* ws, size_t ws_bytes, void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!q_win_host || !k_host || !v_host || !head_w_host || !sens_host || !k_out_host || !v_out_host ||
      !indices_host || !budgets_host || !offsets_host)
    return CKV_ERR_INVALID_ARG;
  const Staging g = staging_layout(*shape, *params);
  if (!staging || !aligned(staging, 256) || staging_bytes < g.total) return CKV_ERR_WORKSPACE;
  CKV_TRY(check_ws(shape, params, ws, ws_bytes));
  ckv_shape s = *shape;  // dense device copies
  s.q_stride_row = s.head_dim;
  s.q_stride_head = (int64_t)s.window * s.head_dim;
  s.q_stride_unit = (int64_t)s.n_q_heads * s.q_stride_head;
  s.kv_stride_tok = s.head_dim;
  s.kv_stride_head = (int64_t)s.seq_len * s.head_dim;
  s.kv_stride_unit = (int64_t)s.n_kv_heads * s.kv_stride_head;
  ckv_params p = *params;
  p.head_w_stride_unit = params->head_w_stride_unit ? s.n_q_heads : 0;
  p.sens_stride_unit = params->sens_stride_unit ? params->n_buckets : 0;
  char* d = (char*)staging;
  cudaStream_t st = (cudaStream_t)stream;
  CKV_CUDA(cudaMemcpyAsync(d + g.q, q_win_host, g.q_b, cudaMemcpyHostToDevice, st));
  CKV_CUDA(cudaMemcpyAsync(d + g.k, k_host, g.kv_b, cudaMemcpyHostToDevice, st));
  // The values are only gathered (unless the value-norm ratio streams them): where the device can read the host
  // buffer in place, the gather fetches the kept rows from there and the other 98 % of V never cross the bus.
  const void* v_dev = params->value_norm ? nullptr : mapped_host_pointer(v_host);
  if (!v_dev) {
    CKV_CUDA(cudaMemcpyAsync(d + g.v, v_host, g.kv_b, cudaMemcpyHostToDevice, st));
    v_dev = d + g.v;
  }
  CKV_CUDA(cudaMemcpyAsync(d + g.head_w, head_w_host, g.hw_b, cudaMemcpyHostToDevice, st));
  CKV_CUDA(cudaMemcpyAsync(d + g.sens, sens_host, g.sens_b, cudaMemcpyHostToDevice, st));
  if (params->gate_coords) {
    CKV_CUDA(cudaMemcpyAsync(d + g.coords, params->gate_coords, g.coords_b, cudaMemcpyHostToDevice, st));
    p.gate_coords = reinterpret_cast<const int32_t*>(d + g.coords);
  }
  CKV_TRY(ckv_compress(&s, &p, d + g.q, d + g.k, v_dev, (const float*)(d + g.head_w), (const float*)(d + g.sens),
                       d + g.k_out, d + g.v_out, (int32_t*)(d + g.indices), (int32_t*)(d + g.budgets),
                       (int32_t*)(d + g.offsets), nullptr, nullptr, nullptr, ws, ws_bytes, stream));
  CKV_CUDA(cudaMemcpyAsync(k_out_host, d + g.k_out, g.out_b, cudaMemcpyDeviceToHost, st));
  CKV_CUDA(cudaMemcpyAsync(v_out_host, d + g.v_out, g.out_b, cudaMemcpyDeviceToHost, st));
  CKV_CUDA(cudaMemcpyAsync(indices_host, d + g.indices, g.idx_b, cudaMemcpyDeviceToHost, st));
  CKV_CUDA(cudaMemcpyAsync(budgets_host, d + g.budgets, g.bud_b, cudaMemcpyDeviceToHost, st));
  CKV_CUDA(cudaMemcpyAsync(offsets_host, d + g.offsets, g.off_b, cudaMemcpyDeviceToHost, st));
  CKV_CUDA(cudaStreamSynchronize(st));
  return CKV_OK;
}

ckv_status ckv_device_status(const void* ws, void* stream) {
  if (!ws) {   // the fixed scratch of ckv_score_noalloc on the current device
    char* scratch = nullptr;
    if (noalloc_scratch(&scratch) != CKV_OK) return CKV_ERR_CUDA;
    ws = scratch;
  }
  if (!aligned(ws, 256)) return CKV_ERR_WORKSPACE;
  int32_t words[2] = {0, 0};   // the code, and the magic word that says the code is meaningful
  cudaStream_t st = (cudaStream_t)stream;
  const char* base = static_cast<const char*>(ws);
  if (cudaMemcpyAsync(&words[0], base, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(&words[1], base + kStatusMagicWord * sizeof(int32_t), sizeof(int32_t), cudaMemcpyDeviceToHost,
                      st) != cudaSuccess)
    return CKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return CKV_ERR_CUDA;
  if (words[1] != kStatusMagic || words[0] == 0) return CKV_OK;   // never used by a call, or nothing recorded
  // a recorded code is reported once: clear it (and the words that name the waits) for the calls that follow
  if (cudaMemsetAsync(const_cast<char*>(base), 0, 8 * sizeof(int32_t), st) != cudaSuccess) return CKV_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return CKV_ERR_CUDA;
  return CKV_ERR_TIMEOUT;
}

int ckv_set_score_path(int path) {
  if (path < 0 || path > 2) return -1;
  return g_score_path.exchange(path, std::memory_order_relaxed);
}

void ckv_set_scan_events(void* start_event, void* stop_event) {
  t_scan_start = (cudaEvent_t)start_event;
  t_scan_stop = (cudaEvent_t)stop_event;
}

int ckv_set_tunable(const char* name, int value) {
  if (!name) return -1;
  if (std::string(name) == "group_fuse") return g_group_fuse.exchange(value != 0 ? 1 : 0);
  if (std::string(name) == "pdl") return g_pdl.exchange(value != 0 ? 1 : 0);
  if (std::string(name) == "run_tiles") return value >= 1 && value <= 64 ? g_run_tiles.exchange(value) : -1;
  if (std::string(name) == "l2_hints") return value == 0 || value == 1 ? g_l2_hints.exchange(value) : -1;
  if (std::string(name) == "wait_limit_us") {
    if (value < 1) return -1;
    return (int)(g_wait_limit_ns.exchange((unsigned long long)value * 1000ull) / 1000ull);
  }
  return -1;
}

int64_t ckv_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int ckv_gate_depth_map_host(const float* src, int n_src, int n_dst, int64_t row_elems, float* dst) {
  if (!src || !dst || n_src < 1 || n_dst < 1 || row_elems < 1) return 1;
  for (int l = 0; l < n_dst; ++l) {
    // position of target layer l on the source's layer axis, by relative depth
    const double pos = n_dst > 1 ? (double)l * (n_src - 1) / (double)(n_dst - 1) : 0.0;
    const int below = std::min((int)pos, n_src - 1), above = std::min(below + 1, n_src - 1);
    const double frac = pos - below;
    const float* a = src + (int64_t)below * row_elems;
    const float* b = src + (int64_t)above * row_elems;
    float* out = dst + (int64_t)l * row_elems;
    for (int64_t c = 0; c < row_elems; ++c) out[c] = (float)((double)a[c] * (1.0 - frac) + (double)b[c] * frac);
  }
  return 0;
}

const char* ckv_status_string(ckv_status status) {
  switch (status) {
    case CKV_OK: return "ok";
    case CKV_ERR_INVALID_ARG: return "invalid argument";
    case CKV_ERR_UNSUPPORTED: return "unsupported shape";
    case CKV_ERR_WORKSPACE: return "work space missing, misaligned or too small";
    case CKV_ERR_CUDA: return "CUDA error";
    case CKV_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

int ckv_version(void) { return 100; }

// Host-only check of the budget split used by the device code (same source, compiled for the host).
int ckv_allocate_rows_host(int hkv, int64_t n, int64_t f, int64_t P, const int64_t* demands, int64_t* out) {
  if (hkv < 1 || hkv > kMaxKvHeads) return 1;
  long long dem[kMaxKvHeads], e[kMaxKvHeads];
  for (int g = 0; g < hkv; ++g) dem[g] = demands[g];
  if (!allocate_rows(hkv, n, f, P, dem, e)) return 2;
  for (int g = 0; g < hkv; ++g) out[g] = e[g];
  return 0;
}

}  // extern "C"
#pragma GCC visibility pop

// ---------------------------------------------------------------------------------------------
// Scratch for ckv_score_noalloc: a fixed array in every device's global memory, present from the
// moment the library is loaded on that device until the process exits.  Host code must never hand
// the symbol itself to a kernel (on the host the name is only a stand-in); it asks the runtime for
// the device address once per device and passes that.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CKV_NOALLOC_SCRATCH_BYTES];

namespace ckv {
static std::mutex g_noalloc_mutex;
static void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the fixed scratch on the current device (looked up on first use per device).
static ckv_status noalloc_scratch(char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CKV_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return CKV_ERR_CUDA;
    g_noalloc_ptr[dev] = p;
  }
  *out = static_cast<char*>(g_noalloc_ptr[dev]);
  return CKV_OK;
}
}  // namespace ckv

#pragma GCC visibility push(default)
extern "C" ckv_status ckv_score_noalloc(const ckv_shape* shape, const ckv_params* params, const void* q_win,
                                        const void* k, const float* head_w, float* scores, float* colmass,
                                        void* stream) {
  CKV_TRY(check_shape(shape));
  CKV_TRY(check_params(shape, params));
  const TuningScope tuning_scope(*params);
  if (!all_aligned16({q_win, k}) || !all_aligned4({head_w, scores, colmass})) return CKV_ERR_INVALID_ARG;
  if (ws_layout(*shape, *params).score_extent > (size_t)CKV_NOALLOC_SCRATCH_BYTES) return CKV_ERR_WORKSPACE;
  char* scratch = nullptr;
  CKV_TRY(noalloc_scratch(&scratch));
  // score_impl clears the scan's counters before its kernels read them and touches nothing beyond the score
  // stage's sections; the rest of those is written before it is read, so what the previous call left behind
  // is harmless.
  return score_impl(*shape, *params, q_win, k, head_w, scores, colmass, scratch, (cudaStream_t)stream);
}
#pragma GCC visibility pop
