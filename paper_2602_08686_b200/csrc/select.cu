// Per-head exact Top-k (Eq. 8's Top-B branch): a most-significant-digit radix select finds the
// key of the k-th largest score, then one ordered compaction writes the kept positions in
// ascending order; equal scores are resolved toward the lowest index, and the observation window
// is appended.  One CTA per (unit, KV head); integer work only, bit-exact and deterministic.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 1024;

// Order-preserving map from float bits to unsigned: larger float <=> larger key.
__device__ __forceinline__ uint32_t key_of(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(kThreads) select_kernel(ckv_shape s, const float* __restrict__ scores,
                                                          const int32_t* __restrict__ budgets,
                                                          const int32_t* __restrict__ offsets,
                                                          int32_t* __restrict__ indices) {
  __shared__ int hist[256];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_want;
  __shared__ int warp_gt[kThreads / 32], warp_eq[kThreads / 32];
  const int Hkv = s.n_kv_heads, W = s.window, n = s.seq_len - W;
  const int u = blockIdx.x / Hkv, g = blockIdx.x % Hkv;
  const int e = budgets[(int64_t)u * Hkv + g] - W;
  const int64_t rows_per_unit = offsets[(int64_t)u * (Hkv + 1) + Hkv];
  int32_t* out = indices + (int64_t)u * rows_per_unit + offsets[(int64_t)u * (Hkv + 1) + g];
  const float* sc = scores + ((int64_t)u * Hkv + g) * n;

  for (int i = threadIdx.x; i < W; i += kThreads) out[e + i] = n + i;
  if (e <= 0) return;
  if (e >= n) {
    for (int t = threadIdx.x; t < n; t += kThreads) out[t] = t;
    return;
  }

  // radix select, 8 bits per pass from the top: after the loop `prefix` is the key of the e-th
  // largest score and `want` the number of scores equal to it that are kept
  uint32_t prefix = 0, mask = 0;
  int want = e;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (threadIdx.x < 256) hist[threadIdx.x] = 0;
    __syncthreads();
    for (int t = threadIdx.x; t < n; t += kThreads) {
      const uint32_t key = key_of(sc[t]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xff], 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int acc = 0, dgt = 255;
      for (; dgt > 0; --dgt) {
        if (acc + hist[dgt] >= want) break;
        acc += hist[dgt];
      }
      sh_prefix = prefix | ((uint32_t)dgt << shift);
      sh_want = want - acc;
    }
    __syncthreads();
    prefix = sh_prefix;
    want = sh_want;
    mask |= 0xffu << shift;
    __syncthreads();
  }

  // ordered compaction: thread i owns the contiguous positions [i*chunk, (i+1)*chunk)
  const int chunk = (n + kThreads - 1) / kThreads;
  const int t0 = min(threadIdx.x * chunk, n), t1 = min(t0 + chunk, n);
  int gt = 0, eq = 0;
  for (int t = t0; t < t1; ++t) {
    const uint32_t key = key_of(sc[t]);
    gt += key > prefix;
    eq += key == prefix;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int gt_inc = gt, eq_inc = eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, gt_inc, o), b = __shfl_up_sync(0xffffffffu, eq_inc, o);
    if (lane >= o) gt_inc += a, eq_inc += b;
  }
  if (lane == 31) warp_gt[warp] = gt_inc, warp_eq[warp] = eq_inc;
  __syncthreads();
  if (warp == 0) {
    int a = warp_gt[lane], b = warp_eq[lane];
    int ai = a, bi = b;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, ai, o), y = __shfl_up_sync(0xffffffffu, bi, o);
      if (lane >= o) ai += x, bi += y;
    }
    warp_gt[lane] = ai - a;
    warp_eq[lane] = bi - b;
  }
  __syncthreads();
  int gt_before = warp_gt[warp] + gt_inc - gt, eq_before = warp_eq[warp] + eq_inc - eq;
  for (int t = t0; t < t1; ++t) {
    const uint32_t key = key_of(sc[t]);
    if (key > prefix) {
      out[gt_before + min(eq_before, want)] = t;
      ++gt_before;
    } else if (key == prefix) {
      if (eq_before < want) out[gt_before + eq_before] = t;
      ++eq_before;
    }
  }
}

}  // namespace

cudaError_t launch_select(const ckv_shape& s, const ckv_params&, const float* scores, const int32_t* budgets,
                          const int32_t* offsets, int32_t* indices, cudaStream_t st) {
  select_kernel<<<s.n_units * s.n_kv_heads, kThreads, 0, st>>>(s, scores, budgets, offsets, indices);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
