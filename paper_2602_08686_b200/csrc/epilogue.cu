// Pooling, head-table weighting and group max (Eq. 4's L/W scale, Eq. 6 inside a GQA group), and
// the unit's column mass for the entropy of Eq. 7, in one pass over the per-head column sums.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 256;   // positions per CTA
constexpr int kMaxHalo = 7;     // pool_size <= 15
constexpr int kHeadBatch = 8;   // heads staged in shared memory at a time

// One CTA owns 256 consecutive positions t of one unit and walks over all query heads:
//   scores[u,g,t] = max_{h in g} head_w[h] * pool((L/W) c_h)[t]   for t < n  (pooling never looks past n)
//   colmass[u,t]  = sum_h c_h[t]                                    for t < L  (heads added in index order)
__global__ void __launch_bounds__(kThreads) pool_weight_max_mass(ckv_shape s, ckv_params p,
                                                                 const float* __restrict__ csum,
                                                                 const float* __restrict__ head_w,
                                                                 float* __restrict__ scores,
                                                                 float* __restrict__ colmass) {
  __shared__ float tile[kHeadBatch][kThreads + 2 * kMaxHalo];
  const int L = s.seq_len, n = L - s.window, H = s.n_q_heads, G = H / s.n_kv_heads;
  const int u = blockIdx.y, t0 = blockIdx.x * kThreads, t = t0 + threadIdx.x;
  const int r = (p.pool_kind == CKV_POOL_NONE) ? 0 : p.pool_size / 2;
  const bool avg = p.pool_kind == CKV_POOL_AVG && r > 0;
  const float pad = avg ? 0.f : -INFINITY;   // AVG counts outside positions as zeros, MAX ignores them
  const float scale = (float)L / (float)s.window;
  const float inv_size = 1.f / (float)p.pool_size;
  const float* hw = head_w + (int64_t)u * p.head_w_stride_unit;
  float mass = 0.f, best = -INFINITY;
  for (int h0 = 0; h0 < H; h0 += kHeadBatch) {
    const int nh = min(kHeadBatch, H - h0);
    __syncthreads();
    for (int e = threadIdx.x; e < nh * (kThreads + 2 * r); e += kThreads) {
      const int hh = e / (kThreads + 2 * r), i = e - hh * (kThreads + 2 * r);
      const int tt = t0 - r + i;
      const float* c = csum + ((int64_t)u * H + h0 + hh) * L;
      // positions inside [0, L) are loaded as they are (the mass needs the window columns too);
      // the pooling below replaces what lies outside the prefix by the pad value
      tile[hh][i] = (tt >= 0 && tt < L) ? c[tt] : 0.f;
    }
    __syncthreads();
    for (int hh = 0; hh < nh; ++hh) {
      const int h = h0 + hh;
      const float* row = tile[hh] + threadIdx.x;   // row[i] = c_h[t - r + i]
      if (t < L) mass += row[r];
      if (t < n) {
        float v;
        if (avg) {
          float acc = 0.f;
          for (int i = 0; i <= 2 * r; ++i) {
            const int tt = t - r + i;
            acc += (tt >= 0 && tt < n) ? row[i] : pad;
          }
          v = acc * scale * inv_size;
        } else {
          float m = -INFINITY;
          for (int i = 0; i <= 2 * r; ++i) {
            const int tt = t - r + i;
            m = fmaxf(m, (tt >= 0 && tt < n) ? row[i] : pad);
          }
          v = m * scale;
        }
        best = fmaxf(best, hw[h] * v);
      }
      if ((h + 1) % G == 0) {  // last head of its KV group
        if (t < n) scores[((int64_t)u * s.n_kv_heads + h / G) * n + t] = best;
        best = -INFINITY;
      }
    }
  }
  if (t < L) colmass[(int64_t)u * L + t] = mass;
}

}  // namespace

cudaError_t launch_epilogue(const ckv_shape& s, const ckv_params& p, const float* csum, const float* head_w,
                            float* scores, float* colmass, cudaStream_t st) {
  dim3 grid((s.seq_len + kThreads - 1) / kThreads, s.n_units);
  pool_weight_max_mass<<<grid, kThreads, 0, st>>>(s, p, csum, head_w, scores, colmass);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
