// Risk coordinate (entropy of the unit's normalised window mass, Eq. 7), threshold lookup
// (Alg. 1 (D)), candidate counts (Eq. 8's candidate set) and the clamp of the per-head budgets to
// the unit's total.  One CTA per unit; every reduction adds in a fixed order.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 1024;

__device__ double block_sum(double v, double* sh) {
  sh[threadIdx.x] = v;
  __syncthreads();
  for (int o = kThreads / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  const double r = sh[0];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kThreads) budget_kernel(ckv_shape s, ckv_params p,
                                                          const float* __restrict__ scores,
                                                          const float* __restrict__ colmass,
                                                          const float* __restrict__ sens,
                                                          int32_t* __restrict__ budgets,
                                                          int32_t* __restrict__ offsets,
                                                          int32_t* __restrict__ bucket_out,
                                                          float* __restrict__ entropy_out) {
  __shared__ double sh[kThreads];
  __shared__ int cnt[kMaxKvHeads];
  __shared__ float tau_s;
  const int u = blockIdx.x, L = s.seq_len, W = s.window, n = L - W, Hkv = s.n_kv_heads;

  // entropy of p[t] = colmass[t] / (W H)
  const double norm = 1.0 / ((double)W * (double)s.n_q_heads);
  double acc = 0.0;
  for (int t = threadIdx.x; t < L; t += kThreads) {
    const double pt = (double)colmass[(int64_t)u * L + t] * norm;
    if (pt > 0.0) acc -= pt * log(pt);
  }
  const double ent = block_sum(acc, sh);
  if (threadIdx.x == 0) {
    const double hn = L > 1 ? ent / log((double)L) : 0.0;
    int b = (int)floor(hn * (double)p.n_buckets);
    b = min(max(b, 0), p.n_buckets - 1);
    if (p.bucket_override >= 0) b = min(p.bucket_override, p.n_buckets - 1);
    tau_s = sens[(int64_t)u * p.sens_stride_unit + b];
    if (bucket_out) bucket_out[u] = b;
    if (entropy_out) entropy_out[u] = (float)ent;
  }
  if (threadIdx.x < kMaxKvHeads) cnt[threadIdx.x] = 0;
  __syncthreads();
  const float tau = tau_s;

  // candidate counts (integer sums: order does not matter)
  for (int g = 0; g < Hkv; ++g) {
    const float* sc = scores + ((int64_t)u * Hkv + g) * n;
    int c = 0;
    for (int t = threadIdx.x; t < n; t += kThreads) c += (sc[t] >= tau) ? 1 : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(&cnt[g], c);
  }
  __syncthreads();

  if (threadIdx.x == 0) {
    long long dem[kMaxKvHeads], e[kMaxKvHeads];
    const long long f = p.floor_per_head, B = p.budget_per_head;
    if (B >= L) {
      for (int g = 0; g < Hkv; ++g) e[g] = n;
    } else {
      const long long lo = f > 1 ? f : 1;
      for (int g = 0; g < Hkv; ++g) {
        long long c = cnt[g];
        dem[g] = c < lo ? lo : (c > n ? n : c);
      }
      if (!allocate_rows(Hkv, n, f, (long long)Hkv * (B - W), dem, e))
        for (int g = 0; g < Hkv; ++g) e[g] = B - W;  // unreachable for validated arguments
    }
    int off = 0;
    for (int g = 0; g < Hkv; ++g) {
      budgets[(int64_t)u * Hkv + g] = (int)e[g] + W;
      offsets[(int64_t)u * (Hkv + 1) + g] = off;
      off += (int)e[g] + W;
    }
    offsets[(int64_t)u * (Hkv + 1) + Hkv] = off;
  }
}

}  // namespace

cudaError_t launch_budget(const ckv_shape& s, const ckv_params& p, const float* scores, const float* colmass,
                          const float* sens, int32_t* budgets, int32_t* offsets, int32_t* bucket, float* entropy,
                          cudaStream_t st) {
  budget_kernel<<<s.n_units, kThreads, 0, st>>>(s, p, scores, colmass, sens, budgets, offsets, bucket, entropy);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
