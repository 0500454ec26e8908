// Risk coordinate (entropy of the unit's normalised window mass, Eq. 7), threshold lookup
// (Alg. 1 (D)), candidate counts (Eq. 8's candidate set) and the clamp of the per-head budgets to
// the unit's total.  One launch of counting CTAs; the last one of a unit to finish splits the rows.
// The entropy arrives as per-block partial sums, added here in a fixed order; the counts are integers.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 256;
constexpr int kPerThread = kCountSpan / kThreads;

// allocate_rows with the CTA's threads: the same split, found by the same rules.  Heads are ranked by
// counting (stable, like the insertion sort), every (a, b) is tested by some thread and the first
// consistent pair in the order of the serial loops wins, the shares and the ranking of the remainders
// are one head per thread.  dem and e live in shared memory; every thread of the CTA must call.
__device__ bool allocate_rows_cta(int hkv, long long n, long long f, long long P, const long long* dem,
                                  long long* e) {
  __shared__ int order[kMaxKvHeads];
  __shared__ long long low[kMaxKvHeads + 1], high[kMaxKvHeads + 1], rem[kMaxKvHeads];
  __shared__ int best;
  const int tid = threadIdx.x;
  if (tid < hkv) {
    int rank = 0;
    for (int j = 0; j < hkv; ++j) rank += (dem[j] < dem[tid] || (dem[j] == dem[tid] && j < tid)) ? 1 : 0;
    order[rank] = tid;
  }
  if (tid == 0) best = 0x7fffffff;
  __syncthreads();
  if (tid <= hkv) {   // sums of the tid smallest and of the tid largest demands
    long long lo = 0, hi = 0;
    for (int r = 0; r < tid; ++r) lo += dem[order[r]], hi += dem[order[hkv - 1 - r]];
    low[tid] = lo, high[tid] = hi;
  }
  __syncthreads();
  const long long total = low[hkv];
  for (int idx = tid; idx < (hkv + 1) * (hkv + 1); idx += blockDim.x) {
    const int a = idx / (hkv + 1), b = idx - a * (hkv + 1);
    if (a + b > hkv) continue;
    const long long R = P - a * f - b * n, D = total - low[a] - high[b];
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
    if (ok) atomicMin(&best, idx);
  }
  __syncthreads();
  if (best == 0x7fffffff) return false;
  const int a = best / (hkv + 1), b = best - a * (hkv + 1), mid = hkv - a - b;
  const long long R = P - a * f - b * n, D = total - low[a] - high[b];
  if (tid < hkv) {   // tid is a rank here
    const int g = order[tid];
    if (tid < a) e[g] = f, rem[g] = 0;
    else if (tid >= hkv - b) e[g] = n, rem[g] = 0;
    else e[g] = (R * dem[g]) / D, rem[g] = (R * dem[g]) % D;
  }
  __syncthreads();
  long long left = 0;
  if (mid > 0) {
    left = R;
    for (int r = a; r < hkv - b; ++r) left -= e[order[r]];
  }
  bool more = false;
  if (tid < hkv && rem[tid] > 0) {   // the `left` largest remainders get one more row, ties to the lowest head
    int rr = 0;
    for (int j = 0; j < hkv; ++j) rr += (rem[j] > rem[tid] || (rem[j] == rem[tid] && j < tid)) ? 1 : 0;
    more = rr < left;
  }
  __syncthreads();   // every thread has read e and rem
  if (more) e[tid] += 1;
  __syncthreads();
  return true;
}

// CTA (g * S + slice, u) counts the candidates of one slice of one KV head.
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
  __shared__ long long dem_s[kMaxKvHeads], e_s[kMaxKvHeads];
  __shared__ int raw_s;   // candidates of head 0 (the shared elastic selection gives every head the same scores)
  pdl_launch_dependents();
  pdl_wait();   // scores and entropy partials come from the kernel before
  const int u = blockIdx.y, L = s.seq_len, W = s.window, n = L - W, Hkv = s.n_kv_heads;
  const int g = blockIdx.x / S, slice = blockIdx.x - g * S;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // the scores first: their latency covers the threshold lookup
  const float* sc = scores + ((int64_t)u * Hkv + g) * n;
  float x[kPerThread];
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int t = slice * kCountSpan + i * kThreads + (int)threadIdx.x;
    x[i] = t < n ? sc[t] : -INFINITY;
  }
  if (warp == 0) {
    // lane l adds the partials l, l + 32, ... in order, then a shuffle tree: the same sum in every CTA
    double ent = 0.0;
    for (int b = lane; b < nblk; b += 32) ent += ent_part[(int64_t)u * nblk + b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ent += __shfl_xor_sync(0xffffffffu, ent, o);
    if (lane == 0) {
      const double hn = L > 1 ? ent / log((double)L) : 0.0;
      int b = (int)floor(hn * (double)p.n_buckets);
      b = min(max(b, 0), p.n_buckets - 1);
      if (p.bucket_override >= 0) b = min(p.bucket_override, p.n_buckets - 1);
      if (p.gate_coords) {   // Alg. 1 (D): tau = T_gate[l, b_ent, b_ppl, B_l]; coordinates held inside the table
        const int32_t* c = p.gate_coords + (int64_t)u * 3;
        const int l = min(max(c[0], 0), p.n_gate_layers - 1), bp = min(max(c[1], 0), p.n_ppl_bins - 1);
        const int bb = min(max(c[2], 0), p.n_budget_levels - 1);
        tau_s = sens[(((int64_t)l * p.n_buckets + b) * p.n_ppl_bins + bp) * p.n_budget_levels + bb];
      } else {
        tau_s = sens[(int64_t)u * p.sens_stride_unit + b];
      }
      bucket_s = b, ent_s = ent, cnt_s = 0;
    }
  }
  __syncthreads();
  const float tau = tau_s;
  int c = 0;
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int t = slice * kCountSpan + i * kThreads + (int)threadIdx.x;
    c += (t < n && x[i] >= tau) ? 1 : 0;
  }
  c = __reduce_add_sync(0xffffffffu, c);
  if (lane == 0 && c) atomicAdd(&cnt_s, c);
  __syncthreads();
  if (threadIdx.x == 0) {
    cnt_part[((int64_t)u * Hkv + g) * S + slice] = cnt_s;
    __threadfence();
    last_s = atomicAdd(done + u, 1) == Hkv * S - 1;
  }
  __syncthreads();
  if (!last_s) return;
  __threadfence();
  const long long f = p.floor_per_head, B = p.budget_per_head;
  const long long lowest = f > 1 ? f : 1;
  for (int gg = warp; gg < Hkv; gg += kThreads / 32) {   // a warp per head adds its slices
    int cc = 0;
    for (int sl = lane; sl < S; sl += 32) cc += __ldcg(cnt_part + ((int64_t)u * Hkv + gg) * S + sl);
    cc = __reduce_add_sync(0xffffffffu, cc);
    if (lane == 0) {
      dem_s[gg] = cc < lowest ? lowest : (cc > n ? n : cc);
      if (gg == 0) raw_s = cc;
    }
  }
  __syncthreads();
  if (B >= L) {
    if ((int)threadIdx.x < Hkv) e_s[threadIdx.x] = n;
    __syncthreads();
  } else if (p.shared_elastic) {
    // Eq. 8: all candidates when they fit the budget, else the Top-B of them; the floor still applies
    long long keep = raw_s < B - W ? raw_s : B - W;
    keep = keep < f ? f : keep;
    keep = keep > n ? n : keep;
    if ((int)threadIdx.x < Hkv) e_s[threadIdx.x] = keep;
    __syncthreads();
  } else if (!allocate_rows_cta(Hkv, n, f, (long long)Hkv * (B - W), dem_s, e_s)) {
    if ((int)threadIdx.x < Hkv) e_s[threadIdx.x] = B - W;  // unreachable for validated arguments
    __syncthreads();
  }
  if (threadIdx.x != 0) return;
  done[u] = 0;   // ready for the next call on this work space
  const long long* e = e_s;
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

// Eq. 6 over all heads of the unit: every KV head's score row becomes the maximum over the unit's rows.
__global__ void __launch_bounds__(kThreads) unit_max_kernel(ckv_shape s, float* __restrict__ scores) {
  const int u = blockIdx.y, Hkv = s.n_kv_heads, n = s.seq_len - s.window;
  const int t = blockIdx.x * kThreads + threadIdx.x;
  if (t >= n) return;
  float* row = scores + (int64_t)u * Hkv * n + t;
  float m = row[0];
  for (int g = 1; g < Hkv; ++g) m = fmaxf(m, row[(int64_t)g * n]);
  for (int g = 0; g < Hkv; ++g) row[(int64_t)g * n] = m;
}

}  // namespace

cudaError_t launch_unit_max(const ckv_shape& s, float* scores, cudaStream_t st) {
  const int n = s.seq_len - s.window;
  if (n <= 0 || s.n_kv_heads < 2) return cudaSuccess;
  unit_max_kernel<<<dim3((n + kThreads - 1) / kThreads, s.n_units), kThreads, 0, st>>>(s, scores);
  count_launch();
  return cudaGetLastError();
}

BudgetLayout budget_layout(const ckv_shape& s) {
  BudgetLayout b{};
  b.nblk = (s.seq_len + kEntSpan - 1) / kEntSpan;
  const int n = s.seq_len - s.window;
  b.S = n > 0 ? (n + kCountSpan - 1) / kCountSpan : 1;
  const int64_t heads = (int64_t)s.n_units * s.n_kv_heads;
  b.ent_bytes = (size_t)s.n_units * b.nblk * sizeof(double);
  b.cnt_bytes = (size_t)heads * b.S * sizeof(int);
  b.done_bytes = (size_t)s.n_units * sizeof(int);
  return b;
}

cudaError_t launch_budget(const ckv_shape& s, const ckv_params& p, const float* scores, const float* sens,
                          int32_t* budgets, int32_t* offsets, int32_t* bucket, float* entropy, void* ent_part,
                          void* cnt_part, void* done, cudaStream_t st) {
  const BudgetLayout b = budget_layout(s);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(s.n_kv_heads * b.S, s.n_units), cfg.blockDim = dim3(kThreads), cfg.stream = st;
  cudaLaunchAttribute attr = pdl_attribute();
  cfg.attrs = &attr, cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, count_allocate, s, p, b.S, b.nblk, scores, sens,
                                           (const double*)ent_part, (int*)cnt_part, (int*)done, budgets, offsets,
                                           bucket, entropy);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ckv
