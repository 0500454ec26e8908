// Per-head exact Top-k (Eq. 8's Top-B branch): a most-significant-digit radix select finds the
// key of the k-th largest score, then one ordered compaction writes the kept positions in
// ascending order; equal scores are resolved toward the lowest index, and the observation window
// is appended.  One CTA per (unit, KV head); integer work only, bit-exact and deterministic.
// Thread i owns the contiguous positions [i*chunk, (i+1)*chunk); when a head's prefix fits
// (chunk <= 32) the keys stay in registers for all four digit passes and the compaction.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kCache = 32;   // keys a thread can keep in registers

// Order-preserving map from float bits to unsigned: larger float <=> larger key.
__device__ __forceinline__ uint32_t key_of(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

template <bool kCached>
__global__ void __launch_bounds__(kThreads) select_kernel(ckv_shape s, const float* __restrict__ scores,
                                                          const int32_t* __restrict__ budgets,
                                                          const int32_t* __restrict__ offsets,
                                                          int32_t* __restrict__ indices) {
  __shared__ int whist[kWarps][256];   // one histogram per warp: no contention between warps
  __shared__ int totals[256];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_want;
  __shared__ int warp_gt[kWarps], warp_eq[kWarps];
  const int Hkv = s.n_kv_heads, W = s.window, n = s.seq_len - W;
  const int u = blockIdx.x / Hkv, g = blockIdx.x % Hkv;
  const int e = budgets[(int64_t)u * Hkv + g] - W;
  const int64_t rows_per_unit = offsets[(int64_t)u * (Hkv + 1) + Hkv];
  int32_t* out = indices + (int64_t)u * rows_per_unit + offsets[(int64_t)u * (Hkv + 1) + g];
  const float* sc = scores + ((int64_t)u * Hkv + g) * n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  for (int i = threadIdx.x; i < W; i += kThreads) out[e + i] = n + i;
  if (e <= 0) return;
  if (e >= n) {
    for (int t = threadIdx.x; t < n; t += kThreads) out[t] = t;
    return;
  }

  const int chunk = (n + kThreads - 1) / kThreads;
  const int t0 = min(threadIdx.x * chunk, n), t1 = min(t0 + chunk, n);
  uint32_t keys[kCached ? kCache : 1];
  if (kCached) {
#pragma unroll
    for (int j = 0; j < kCache; ++j) keys[j] = (t0 + j < t1) ? key_of(sc[t0 + j]) : 0u;
  }

  // radix select, 8 bits per pass from the top: after the loop `prefix` is the key of the e-th
  // largest score and `want` the number of scores equal to it that are kept
  uint32_t prefix = 0, mask = 0;
  int want = e;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = lane; i < 256; i += 32) whist[warp][i] = 0;
    __syncwarp();
    // consecutive equal digits of a thread are added in one go (scores of one head share their top bits)
    int run_bin = -1, run_cnt = 0;
#pragma unroll
    for (int j = 0; j < (kCached ? kCache : 1); ++j) {
      if (kCached) {
        if (t0 + j < t1 && (keys[j] & mask) == prefix) {
          const int bin = (keys[j] >> shift) & 0xff;
          if (bin == run_bin) {
            ++run_cnt;
          } else {
            if (run_cnt) atomicAdd(&whist[warp][run_bin], run_cnt);
            run_bin = bin, run_cnt = 1;
          }
        }
      }
    }
    if (!kCached) {
      for (int t = t0; t < t1; ++t) {
        const uint32_t key = key_of(sc[t]);
        if ((key & mask) == prefix) {
          const int bin = (key >> shift) & 0xff;
          if (bin == run_bin) {
            ++run_cnt;
          } else {
            if (run_cnt) atomicAdd(&whist[warp][run_bin], run_cnt);
            run_bin = bin, run_cnt = 1;
          }
        }
      }
    }
    if (run_cnt) atomicAdd(&whist[warp][run_bin], run_cnt);
    __syncthreads();
    // 256 threads add the per-warp histograms, then warp 0 (lane i owns digits 8 i .. 8 i + 7) finds the
    // digit d with count(digit > d) < want <= count(digit >= d)
    if (threadIdx.x < 256) {
      int tot = 0;
#pragma unroll 8
      for (int w = 0; w < kWarps; ++w) tot += whist[w][threadIdx.x];
      totals[threadIdx.x] = tot;
    }
    __syncthreads();
    if (warp == 0) {
      int cnt[8], mine = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) cnt[e] = totals[8 * lane + e], mine += cnt[e];
      // above = number of matching keys in the digits of higher lanes
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += x;
      }
      int above = incl - mine;
      if (above < want && incl >= want) {   // the digit lies in this lane's range: exactly one lane
        int dgt = 7;
        for (; dgt > 0; --dgt) {
          if (above + cnt[dgt] >= want) break;
          above += cnt[dgt];
        }
        sh_prefix = prefix | ((uint32_t)(8 * lane + dgt) << shift);
        sh_want = want - above;
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    want = sh_want;
    mask |= 0xffu << shift;
    __syncthreads();
  }

  // ordered compaction
  int gt = 0, eq = 0;
  if (kCached) {
#pragma unroll
    for (int j = 0; j < kCache; ++j)
      if (t0 + j < t1) gt += keys[j] > prefix, eq += keys[j] == prefix;
  } else {
    for (int t = t0; t < t1; ++t) {
      const uint32_t key = key_of(sc[t]);
      gt += key > prefix;
      eq += key == prefix;
    }
  }
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
  auto place = [&](uint32_t key, int t) {
    if (key > prefix) {
      out[gt_before + min(eq_before, want)] = t;
      ++gt_before;
    } else if (key == prefix) {
      if (eq_before < want) out[gt_before + eq_before] = t;
      ++eq_before;
    }
  };
  if (kCached) {
#pragma unroll
    for (int j = 0; j < kCache; ++j)
      if (t0 + j < t1) place(keys[j], t0 + j);
  } else {
    for (int t = t0; t < t1; ++t) place(key_of(sc[t]), t);
  }
}

}  // namespace

cudaError_t launch_select(const ckv_shape& s, const ckv_params&, const float* scores, const int32_t* budgets,
                          const int32_t* offsets, int32_t* indices, cudaStream_t st) {
  const int n = s.seq_len - s.window;
  const int grid = s.n_units * s.n_kv_heads;
  if ((n + kThreads - 1) / kThreads <= kCache)
    select_kernel<true><<<grid, kThreads, 0, st>>>(s, scores, budgets, offsets, indices);
  else
    select_kernel<false><<<grid, kThreads, 0, st>>>(s, scores, budgets, offsets, indices);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
