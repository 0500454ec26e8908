// Prompt-global window mass (Alg. 1 (A)): the paper averages the attention over all layers and heads of a
// prompt before the window sum, so one alpha[t] = (L/W) * mean_{l,h} c_{l,h}[t] and one risk coordinate serve
// all of the prompt's units.  Two small kernels after the scan:
//   prompt_mass    pmass[s,t] = sum over the prompt's local units of colmass[u,t]   (units in index order)
//   global_scores  scores[u,g,t] = (max_{h in g} head_w[h]) * pool(alpha_s)[t],  alpha_s = (L/W) pmass / (N H);
//                  colmass[u,:] <- pmass[s,:] / N, the mass the budget stage takes its entropy from
// N is the number of units of the prompt on ALL devices: when a prompt's layers are spread over several GPUs the
// caller adds the pmass arrays of the ranks (one all-reduce of [prompts, L] floats) between the two kernels.
// alpha >= 0, so Eq. 6's maximum over a group's heads reduces to the group's largest weight.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads) prompt_mass_kernel(int L, int upp, const float* __restrict__ colmass,
                                                               float* __restrict__ pmass) {
  const int s = blockIdx.y, t = blockIdx.x * kThreads + threadIdx.x;
  if (t >= L) return;
  float m = 0.f;
  for (int i = 0; i < upp; ++i) m += colmass[((int64_t)s * upp + i) * L + t];
  pmass[(int64_t)s * L + t] = m;
}

__global__ void __launch_bounds__(kThreads) global_scores_kernel(ckv_shape s, ckv_params p, int units_total,
                                                                 const float* __restrict__ head_w,
                                                                 const float* __restrict__ pmass,
                                                                 float* __restrict__ scores,
                                                                 float* __restrict__ colmass) {
  const int u = blockIdx.z, g = blockIdx.y, t = blockIdx.x * kThreads + threadIdx.x;
  const int L = s.seq_len, n = L - s.window, H = s.n_q_heads, G = H / s.n_kv_heads;
  if (t >= L) return;
  const float* pm = pmass + (int64_t)(u / p.units_per_prompt) * L;
  if (g == 0) colmass[(int64_t)u * L + t] = pm[t] / (float)units_total;
  if (t >= n) return;
  const float* hw = head_w + (int64_t)u * p.head_w_stride_unit + g * G;
  float wmax = hw[0];
  for (int h = 1; h < G; ++h) wmax = fmaxf(wmax, hw[h]);
  const float scale = ((float)L / (float)s.window) / ((float)units_total * (float)H);
  const int r = p.pool_kind == CKV_POOL_NONE ? 0 : p.pool_size / 2;
  float pooled;
  if (p.pool_kind == CKV_POOL_AVG && r > 0) {   // positions outside the prefix count as zeros
    float acc = 0.f;
    for (int i = -r; i <= r; ++i)
      if (t + i >= 0 && t + i < n) acc += pm[t + i] * scale;
    pooled = acc / (float)(2 * r + 1);
  } else {                                        // max (or none): positions outside the prefix are ignored
    pooled = pm[t] * scale;
    for (int i = -r; i <= r; ++i)
      if (t + i >= 0 && t + i < n) pooled = fmaxf(pooled, pm[t + i] * scale);
  }
  scores[((int64_t)u * s.n_kv_heads + g) * n + t] = wmax * pooled;
}

}  // namespace

cudaError_t launch_prompt_mass(const ckv_shape& s, const ckv_params& p, const float* colmass, float* pmass,
                               cudaStream_t st) {
  dim3 grid((s.seq_len + kThreads - 1) / kThreads, s.n_units / p.units_per_prompt);
  prompt_mass_kernel<<<grid, kThreads, 0, st>>>(s.seq_len, p.units_per_prompt, colmass, pmass);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_global_scores(const ckv_shape& s, const ckv_params& p, int units_total, const float* head_w,
                                 const float* pmass, float* scores, float* colmass, cudaStream_t st) {
  dim3 grid((s.seq_len + kThreads - 1) / kThreads, s.n_kv_heads, s.n_units);
  global_scores_kernel<<<grid, kThreads, 0, st>>>(s, p, units_total, head_w, pmass, scores, colmass);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
