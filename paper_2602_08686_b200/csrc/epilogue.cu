// Pooling, head-table weighting and group max (Eq. 4's L/W scale, Eq. 6 inside a GQA group), and
// the unit's column mass for the entropy of Eq. 7.
#include "ckv_common.cuh"

namespace ckv {
namespace {

// scores[u,g,t] = max_{h in g} head_w[h] * pool((L/W) c_h)[t],  t in [0,n)
__global__ void __launch_bounds__(256) pool_weight_max(ckv_shape s, ckv_params p, const float* __restrict__ csum,
                                                       const float* __restrict__ head_w,
                                                       float* __restrict__ scores) {
  const int L = s.seq_len, n = L - s.window, G = s.n_q_heads / s.n_kv_heads;
  const int u = blockIdx.z, g = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const int r = (p.pool_kind == CKV_POOL_NONE) ? 0 : p.pool_size / 2;
  const float scale = (float)L / (float)s.window;
  const float* hw = head_w + (int64_t)u * p.head_w_stride_unit;
  const int lo = max(t - r, 0), hi = min(t + r, n - 1);
  float best = -INFINITY;
  for (int h = g * G; h < (g + 1) * G; ++h) {
    const float* c = csum + ((int64_t)u * s.n_q_heads + h) * L;
    float v;
    if (p.pool_kind == CKV_POOL_AVG && r > 0) {
      float a = 0.f;
      for (int j = lo; j <= hi; ++j) a += c[j];
      v = a * scale / (float)p.pool_size;
    } else {
      float m = c[lo];
      for (int j = lo + 1; j <= hi; ++j) m = fmaxf(m, c[j]);
      v = m * scale;
    }
    best = fmaxf(best, hw[h] * v);
  }
  scores[((int64_t)u * s.n_kv_heads + g) * n + t] = best;
}

// colmass[u,t] = sum_h c_h[t], heads added in index order
__global__ void __launch_bounds__(256) column_mass(ckv_shape s, const float* __restrict__ csum,
                                                   float* __restrict__ colmass) {
  const int L = s.seq_len, u = blockIdx.y;
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= L) return;
  float m = 0.f;
  for (int h = 0; h < s.n_q_heads; ++h) m += csum[((int64_t)u * s.n_q_heads + h) * L + t];
  colmass[(int64_t)u * L + t] = m;
}

}  // namespace

cudaError_t launch_epilogue(const ckv_shape& s, const ckv_params& p, const float* csum, const float* head_w,
                            float* scores, float* colmass, cudaStream_t st) {
  const int n = s.seq_len - s.window;
  if (n > 0) {
    dim3 grid((n + 255) / 256, s.n_kv_heads, s.n_units);
    pool_weight_max<<<grid, 256, 0, st>>>(s, p, csum, head_w, scores);
    count_launch();
  }
  dim3 grid2((s.seq_len + 255) / 256, s.n_units);
  column_mass<<<grid2, 256, 0, st>>>(s, csum, colmass);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
