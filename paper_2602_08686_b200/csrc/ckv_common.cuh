// Internal declarations shared by the translation units of libckv (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ckv.h"

namespace ckv {

constexpr int kHeadDim = 128;
constexpr int kMaxWindow = 64;
constexpr int kMaxKvHeads = 64;
constexpr int kPlainKeysPerBlock = 256;  // keys per CTA in the plain (SIMT) score kernels
constexpr int kEntSpan = 512;            // positions per entropy partial of the budget stage
constexpr int kAttendMaxRows = 32;       // query rows (group size x decode queries) of the decode-side check
constexpr int kVnormRows = 256;          // value rows per block sum of the value-norm stage
constexpr int kCountSpan = 8192;         // scores per counting CTA of the budget stage
constexpr int kMaxDevices = 64;          // devices the per-device caches of the host code cover

// log2(e): the softmax is evaluated in base 2, x = (q.k) * log2(e) / sqrt(d)
constexpr float kLog2e = 1.4426950408889634f;

// Work-space sections (byte offsets from the 256-byte aligned base).
struct WsLayout {
  size_t status;   // 64 x int32: [0] device status word, the rest scheduler counters
  size_t csum;     // float [Nu, H, L]        c_h[t]
  size_t part;     // float2 [Nu, H, W, nblk] per-block (max, sum) of the row statistics
  size_t stat;     // float2 [Nu, H, W]       (row max, row max + log2 row sum), base-2 domain
  size_t colmass;  // float [Nu, L]           used when the caller passes no buffer
  size_t scores;   // float [Nu, Hkv, n]      likewise
  size_t bucket;   // int32 [Nu]
  size_t entropy;  // float [Nu]
  size_t tc_part;  // float2 [C, T+2, 128]     partial row statistics of the tensor-core scan
  size_t tc_stat;  // float2 [C, 128]          final row statistics per chunk
  size_t tc_flags; // int32 [C, 5]             completion counters and ready flags
  size_t ent_part; // double [Nu, nblk]        entropy partials of the budget stage (nblk = ceil(L / kEntSpan))
  size_t cnt_part; // int32 [Nu, Hkv, S]       candidate counts per slice
  size_t bud_done; // int32 [Nu]               CTAs of the unit that have finished counting
  size_t pmass;    // float [Nu / units_per_prompt, L] window mass summed over a prompt's units (only with global_alpha)
  size_t att_ml;   // float2 [Nu, Hkv, slices, 32] and ...
  size_t att_o;    // float [Nu, Hkv, slices, 32, 128]: per-slice partial results of the decode-side check
  size_t vn_part;  // float [Nu, Hkv, ceil(L / kVnormRows)] block sums of the value-row norms
  size_t vn_rho;   // float [Nu, Hkv, L]       value-norm ratios of the fused call (only with value_norm)
  size_t score_extent;  // end of the sections the score stage uses (they come first)
  size_t total;
  int nblk;
};

// Scratch of the budget stage: entropy blocks per unit, score slices per KV head.
struct BudgetLayout {
  int nblk, S;
  size_t ent_bytes, cnt_bytes, done_bytes;
};
BudgetLayout budget_layout(const ckv_shape& s);

// Sizes of the tensor-core scan's scratch for a shape (chunks of 128 query rows x whole key range).
struct TcLayout {
  int RB, T;
  int64_t C;
  size_t part_bytes, stat_bytes, flag_bytes;
};
TcLayout tc_layout(const ckv_shape& s);
bool score_tc_supported(const ckv_shape& s);
// Grouped output of the scan (see score_tc.cu): per KV group the weighted maximum over its query heads and
// their summed column mass, [Nu, Hkv, L] each, instead of the per-head column sums.  Possible when a group's
// heads fill one row block, there are at least two of them and the pooling is max or none; requires
// head weights >= 0 (a maximum commutes with the pooling only then).
struct TcGrouped {
  float* zgrp;
  float* mgrp;
  const float* head_w;
  int64_t hw_stride;
};
bool score_tc_groupable(const ckv_shape& s, const ckv_params& p);
// flags must be zero at launch (tc_layout's flag_bytes).
cudaError_t launch_score_tc(const ckv_shape& s, const void* q, const void* k, float* csum, const TcGrouped* grp,
                            void* part, void* stat, int* flags, int* status, cudaStream_t st);

WsLayout ws_layout(const ckv_shape& s, const ckv_params& p);

void count_launch(int n = 1);
// Time limit of every bounded device-side wait, in nanoseconds (ckv_set_tunable "wait_limit_us"; default 2 s).
unsigned long long wait_limit_ns();

// Programmatic dependent launch between the small kernels that follow the scan: a kernel launched with
// pdl_attribute() may be scheduled while its predecessor in the stream drains, and must call pdl_wait() before it
// touches anything the predecessor wrote (or reads what it will overwrite); a predecessor lets it start early with
// pdl_launch_dependents().  Both are no-ops in a kernel launched the ordinary way.
bool pdl_enabled();
// Scheduling settings of the call in progress on this thread (params->tuning over the process-wide defaults).
int tuning_run_tiles();
int tuning_l2_hints();
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
inline cudaLaunchAttribute pdl_attribute() {
  cudaLaunchAttribute a{};
  a.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  a.val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
  return a;
}

// Launchers; each returns cudaGetLastError() after queuing its kernels.
cudaError_t launch_score_plain(const ckv_shape& s, const void* q, const void* k, float* csum, float2* part,
                               float2* stat, int nblk, cudaStream_t st);
// The epilogue also writes marker_value to *marker (which scan produced the row statistics in the work space),
// leaves the budget stage's entropy partials (one per kEntSpan positions) and clears its
// arrival counters; launch_entropy_partials does the same from a column mass the caller supplies.
cudaError_t launch_epilogue(const ckv_shape& s, const ckv_params& p, const float* csum, const float* head_w,
                            float* scores, float* colmass, void* ent_part, void* done, int* marker, int marker_value,
                            cudaStream_t st);
// The same from the scan's grouped output: pooling of zgrp inside the prefix, column mass from mgrp.
cudaError_t launch_epilogue_grouped(const ckv_shape& s, const ckv_params& p, const float* zgrp, const float* mgrp,
                                    float* scores, float* colmass, void* ent_part, void* done, int* marker,
                                    int marker_value, cudaStream_t st);
cudaError_t launch_entropy_partials(const ckv_shape& s, const float* colmass, void* ent_part, void* done,
                                    cudaStream_t st);
// Expects the entropy partials and cleared counters of one of the two launchers above.
cudaError_t launch_budget(const ckv_shape& s, const ckv_params& p, const float* scores, const float* sens,
                          int32_t* budgets, int32_t* offsets, int32_t* bucket, float* entropy, void* ent_part,
                          void* cnt_part, void* done, cudaStream_t st);
// Value-norm ratio (Eq. 4's rho): row norms and block sums of V, then the division by mean + eps (and the
// multiplication of the prefix scores when given).
cudaError_t launch_vnorm_rows(const ckv_shape& s, const void* v, float* rho, float* part, cudaStream_t st);
cudaError_t launch_vnorm_finish(const ckv_shape& s, float eps, float* rho, const float* part, float* scores,
                                cudaStream_t st);
// Prompt-global alpha (Alg. 1 (A)): per-prompt sums of the units' column mass, then scores from them.
cudaError_t launch_prompt_mass(const ckv_shape& s, const ckv_params& p, const float* colmass, float* pmass,
                               cudaStream_t st);
cudaError_t launch_global_scores(const ckv_shape& s, const ckv_params& p, int units_total, const float* head_w,
                                 const float* pmass, float* scores, float* colmass, cudaStream_t st);
// Kept attention mass of the window rows on the retained set (Prop. 4.1's 1 - m), from the gathered keys and the
// row statistics in the work space; marker tells which scan wrote them (low byte 2: the tensor-core kernel).
constexpr int kPathMarkerWord = 48;   // index into the work space's 64 status words
cudaError_t launch_kept_mass(const ckv_shape& s, const ckv_params& p, const void* q, const void* k_out,
                             const int32_t* indices, const int32_t* budgets, const int32_t* offsets,
                             const void* stat_plain, const void* stat_tc, const int* marker, float* kept,
                             cudaStream_t st);
// Decode-side check: attention of n_dec queries per head over all rows (compressed = 0) or the gathered rows.
int attend_slices(const ckv_shape& s);
cudaError_t launch_attend(const ckv_shape& s, const ckv_params& p, const void* q_dec, int n_dec, const void* k,
                          const void* v, int compressed, const int32_t* budgets, const int32_t* offsets, float* out,
                          float* lse, void* part_ml, void* part_o, cudaStream_t st);
// Eq. 6 over all heads of a unit (the shared elastic selection): scores[u,g,:] <- max_g' scores[u,g',:].
cudaError_t launch_unit_max(const ckv_shape& s, float* scores, cudaStream_t st);
cudaError_t launch_select(const ckv_shape& s, const ckv_params& p, const float* scores, const int32_t* budgets,
                          const int32_t* offsets, int32_t* indices, int* status, cudaStream_t st);
cudaError_t launch_gather(const ckv_shape& s, const ckv_params& p, const void* k, const void* v,
                          const int32_t* indices, const int32_t* offsets, void* k_out, void* v_out,
                          cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Split P prefix rows over `hkv` heads in proportion to demands dem[g] >= 1 with every share held
// in [f, n] (the clamp of the per-head budgets to the unit's total).  Heads are visited in order of
// demand; because the clamp is monotone in the demand, the heads pinned at the floor are the `a`
// smallest demands and the heads pinned at the cap the `b` largest.  All (a, b) are tried until
// the water level R / D of the unpinned heads is consistent with that split.  Shares of unpinned
// heads are rounded down and the remainder goes to the largest fractional parts, ties to the
// lowest head index.  Pure integer arithmetic (products stay below 2^62 for n <= 2^20, hkv <= 64).
// Returns false only if the arguments violate f*hkv <= P <= n*hkv.
__host__ __device__ inline bool allocate_rows(int hkv, long long n, long long f, long long P, const long long* dem,
                                              long long* e) {
  int order[kMaxKvHeads];
  for (int g = 0; g < hkv; ++g) order[g] = g;
  for (int i = 1; i < hkv; ++i) {  // stable insertion sort by demand
    int x = order[i], j = i - 1;
    while (j >= 0 && dem[order[j]] > dem[x]) {
      order[j + 1] = order[j];
      --j;
    }
    order[j + 1] = x;
  }
  long long total = 0;
  for (int g = 0; g < hkv; ++g) total += dem[g];
  long long low_sum = 0;  // sum of the a smallest demands
  for (int a = 0; a <= hkv; ++a) {
    if (a > 0) low_sum += dem[order[a - 1]];
    long long high_sum = 0;
    for (int b = 0; a + b <= hkv; ++b) {
      if (b > 0) high_sum += dem[order[hkv - b]];
      const long long R = P - a * f - b * n;
      const long long D = total - low_sum - high_sum;
      const int mid = hkv - a - b;
      bool ok;
      if (mid == 0) {
        ok = (R == 0);
      } else {
        const long long dmin = dem[order[a]], dmax = dem[order[hkv - b - 1]];
        ok = R >= 0 && R * dmin >= f * D && R * dmax <= n * D;
        if (ok && a > 0) ok = R * dem[order[a - 1]] <= f * D;
        if (ok && b > 0) ok = R * dem[order[hkv - b]] >= n * D;
      }
      if (!ok) continue;
      long long rem[kMaxKvHeads];
      long long given = 0;
      for (int r = 0; r < hkv; ++r) {
        const int g = order[r];
        if (r < a) {
          e[g] = f;
          rem[g] = 0;
        } else if (r >= hkv - b) {
          e[g] = n;
          rem[g] = 0;
        } else {
          e[g] = (R * dem[g]) / D;
          rem[g] = (R * dem[g]) % D;
          given += e[g];
        }
      }
      long long left = mid > 0 ? R - given : 0;
      while (left > 0) {
        int best = -1;
        for (int g = 0; g < hkv; ++g)
          if (rem[g] > 0 && (best < 0 || rem[g] > rem[best])) best = g;
        if (best < 0) return false;
        e[best] += 1;
        rem[best] = 0;
        --left;
      }
      return true;
    }
  }
  return false;
}

}  // namespace ckv
