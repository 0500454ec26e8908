// Risk coordinate (entropy of the unit's normalised window mass, Eq. 7), threshold lookup
// (Alg. 1 (D)), candidate counts (Eq. 8's candidate set) and the clamp of the per-head budgets to
// the unit's total.  Two launches: per-block entropy partials, then counting CTAs of which the last
// one per unit splits the rows.  Every floating-point reduction adds in a fixed order; the counts are
// integers.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 256;
constexpr int kEntPerBlock = 2048;   // positions per CTA of the entropy kernel

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

// ent_part[u, blk] = - sum over the block's positions of p ln p,  p[t] = colmass[t] / (W H)
__global__ void __launch_bounds__(kThreads) entropy_partials(ckv_shape s, const float* __restrict__ colmass,
                                                             double* __restrict__ ent_part, int nblk) {
  __shared__ double sh[kThreads];
  const int u = blockIdx.y, L = s.seq_len;
  const double norm = 1.0 / ((double)s.window * (double)s.n_q_heads);
  const int t0 = blockIdx.x * kEntPerBlock;
  double acc = 0.0;
  for (int i = threadIdx.x; i < kEntPerBlock; i += kThreads) {
    const int t = t0 + i;
    if (t < L) {
      const double pt = (double)colmass[(int64_t)u * L + t] * norm;
      if (pt > 0.0) acc -= pt * log(pt);
    }
  }
  const double tot = block_sum(acc, sh);
  if (threadIdx.x == 0) ent_part[(int64_t)u * nblk + blockIdx.x] = tot;
}

// CTA (g * S + slice, u) counts the candidates of one slice of one KV head; the last CTA of a unit
// to finish adds the counts and splits the unit's rows.
__global__ void __launch_bounds__(kThreads) count_allocate(ckv_shape s, ckv_params p, int S, int nblk,
                                                           const float* __restrict__ scores,
                                                           const float* __restrict__ sens,
                                                           const double* __restrict__ ent_part,
                                                           int* __restrict__ cnt_part, int* __restrict__ done,
                                                           int32_t* __restrict__ budgets,
                                                           int32_t* __restrict__ offsets,
                                                           int32_t* __restrict__ bucket_out,
                                                           float* __restrict__ entropy_out) {
  __shared__ float tau_s;
  __shared__ int bucket_s;
  __shared__ double ent_s;
  __shared__ int cnt_s;
  __shared__ int last_s;
  const int u = blockIdx.y, L = s.seq_len, W = s.window, n = L - W, Hkv = s.n_kv_heads;
  const int g = blockIdx.x / S, slice = blockIdx.x - g * S;
  if (threadIdx.x == 0) {
    double ent = 0.0;
    for (int b = 0; b < nblk; ++b) ent += ent_part[(int64_t)u * nblk + b];   // block order
    const double hn = L > 1 ? ent / log((double)L) : 0.0;
    int b = (int)floor(hn * (double)p.n_buckets);
    b = min(max(b, 0), p.n_buckets - 1);
    if (p.bucket_override >= 0) b = min(p.bucket_override, p.n_buckets - 1);
    tau_s = sens[(int64_t)u * p.sens_stride_unit + b];
    bucket_s = b, ent_s = ent, cnt_s = 0;
  }
  __syncthreads();
  const float tau = tau_s;
  const int per = (n + S - 1) / S;
  const int lo = min(slice * per, n), hi = min(lo + per, n);
  const float* sc = scores + ((int64_t)u * Hkv + g) * n;
  int c = 0;
  for (int t = lo + threadIdx.x; t < hi; t += kThreads) c += (sc[t] >= tau) ? 1 : 0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0 && c) atomicAdd(&cnt_s, c);
  __syncthreads();
  if (threadIdx.x == 0) {
    cnt_part[((int64_t)u * Hkv + g) * S + slice] = cnt_s;
    __threadfence();
    last_s = atomicAdd(done + u, 1) == Hkv * S - 1;
  }
  __syncthreads();
  if (!last_s || threadIdx.x != 0) return;
  __threadfence();
  done[u] = 0;   // ready for the next call on this work space
  long long dem[kMaxKvHeads], e[kMaxKvHeads];
  const long long f = p.floor_per_head, B = p.budget_per_head;
  if (B >= L) {
    for (int gg = 0; gg < Hkv; ++gg) e[gg] = n;
  } else {
    const long long lowest = f > 1 ? f : 1;
    for (int gg = 0; gg < Hkv; ++gg) {
      long long cc = 0;
      for (int sl = 0; sl < S; ++sl) cc += __ldcg(cnt_part + ((int64_t)u * Hkv + gg) * S + sl);
      dem[gg] = cc < lowest ? lowest : (cc > n ? n : cc);
    }
    if (!allocate_rows(Hkv, n, f, (long long)Hkv * (B - W), dem, e))
      for (int gg = 0; gg < Hkv; ++gg) e[gg] = B - W;  // unreachable for validated arguments
  }
  int off = 0;
  for (int gg = 0; gg < Hkv; ++gg) {
    budgets[(int64_t)u * Hkv + gg] = (int)e[gg] + W;
    offsets[(int64_t)u * (Hkv + 1) + gg] = off;
    off += (int)e[gg] + W;
  }
  offsets[(int64_t)u * (Hkv + 1) + Hkv] = off;
  if (bucket_out) bucket_out[u] = bucket_s;
  if (entropy_out) entropy_out[u] = (float)ent_s;
}

}  // namespace

BudgetLayout budget_layout(const ckv_shape& s) {
  BudgetLayout b{};
  b.nblk = (s.seq_len + kEntPerBlock - 1) / kEntPerBlock;
  const int64_t heads = (int64_t)s.n_units * s.n_kv_heads;
  int S = (int)((2 * 148 + heads - 1) / heads);
  b.S = S < 1 ? 1 : (S > 32 ? 32 : S);
  b.ent_bytes = (size_t)s.n_units * b.nblk * sizeof(double);
  b.cnt_bytes = (size_t)heads * b.S * sizeof(int);
  b.done_bytes = (size_t)s.n_units * sizeof(int);
  return b;
}

cudaError_t launch_budget(const ckv_shape& s, const ckv_params& p, const float* scores, const float* colmass,
                          const float* sens, int32_t* budgets, int32_t* offsets, int32_t* bucket, float* entropy,
                          void* ent_part, void* cnt_part, void* done, cudaStream_t st) {
  const BudgetLayout b = budget_layout(s);
  cudaError_t e = cudaMemsetAsync(done, 0, b.done_bytes, st);
  if (e != cudaSuccess) return e;
  entropy_partials<<<dim3(b.nblk, s.n_units), kThreads, 0, st>>>(s, colmass, (double*)ent_part, b.nblk);
  count_allocate<<<dim3(s.n_kv_heads * b.S, s.n_units), kThreads, 0, st>>>(
      s, p, b.S, b.nblk, scores, sens, (const double*)ent_part, (int*)cnt_part, (int*)done, budgets, offsets, bucket,
      entropy);
  count_launch(2);
  return cudaGetLastError();
}

}  // namespace ckv
