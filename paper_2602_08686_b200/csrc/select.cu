// Per-head exact Top-k (Eq. 8's Top-B branch): a most-significant-bit-first search finds the key of
// the k-th largest score, then one ordered compaction writes the kept positions in ascending order;
// equal scores are resolved toward the lowest index, and the observation window is appended.
// One CTA per (unit, KV head); integer work only, bit-exact and deterministic.
// Warp w owns the contiguous positions [w * 32 * chunk, (w + 1) * 32 * chunk) and lane l of it the
// positions w * 32 * chunk + 32 j + l, so that every load is coalesced and a ballot per j gives the
// order inside the warp's range.  When a head's prefix fits (chunk <= 32) the keys stay in registers
// and the search takes one bit per step: count the keys at or above the candidate (a compare per key,
// one warp reduction, one barrier) until the keys that can still be the k-th fit one per thread; these
// are then copied to shared memory and the remaining bits cost one ballot per warp and step.  Longer
// prefixes use 8-bit digits with per-warp histograms and re-read the scores in every pass.
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
  __shared__ int whist[kCached ? 1 : kWarps][256];   // 8-bit path: one histogram per warp
  __shared__ int totals[256];
  __shared__ int wcnt[2][kWarps];
  __shared__ uint32_t list[kCached ? kThreads : 1];   // keys of the narrowed range
  __shared__ int list_fill;
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

  if (threadIdx.x == 0) list_fill = 0;
  for (int i = threadIdx.x; i < W; i += kThreads) out[e + i] = n + i;
  if (e <= 0) return;
  if (e >= n) {
    for (int t = threadIdx.x; t < n; t += kThreads) out[t] = t;
    return;
  }

  const int chunk = (n + kThreads - 1) / kThreads;      // positions per thread
  const int base = warp * 32 * chunk + lane;            // position of (j = 0); (j) is base + 32 j
  const int wend = min((warp + 1) * 32 * chunk, n);     // end of the warp's range
  uint32_t keys[kCached ? kCache : 1];
  if (kCached) {
#pragma unroll
    for (int j = 0; j < kCache; ++j) {
      const int t = base + 32 * j;
      keys[j] = (j < chunk && t < wend) ? key_of(sc[t]) : 0u;   // key 0 is below every real key
    }
  }

  uint32_t prefix = 0;
  int want = e;
  if (kCached) {
    // One bit per step: the k-th largest key is the largest value v with #{keys >= v} >= k.  The keys that
    // can still be the k-th form the range [prefix, prefix + 2^(bit+1)); its size follows from the counts.
    // While the range holds more keys than the CTA has threads, a step compares all cached keys; then the
    // range is copied to shared memory, one key per thread, and the remaining steps cost a ballot each.
    int above = 0;        // keys above the range: at or above every candidate inside it
    int in_range = n;
    int bit = 31, par = 0;
    for (; bit >= 0 && in_range > kThreads; --bit, par ^= 1) {
      const uint32_t cand = prefix | (1u << bit);
      int c[4] = {0, 0, 0, 0};
#pragma unroll
      for (int j = 0; j < kCache; ++j) c[j & 3] += keys[j] >= cand;
      const int cw = __reduce_add_sync(0xffffffffu, (c[0] + c[1]) + (c[2] + c[3]));
      if (lane == 0) wcnt[par][warp] = cw;
      __syncthreads();   // the other buffer is written in the next step, this one again only after that barrier
      const int tot = __reduce_add_sync(0xffffffffu, wcnt[par][lane]);
      if (tot >= e) {
        prefix = cand;
        in_range = tot - above;
      } else {
        in_range -= tot - above;
        above = tot;
      }
    }
    if (bit >= 0) {
      const int sh = bit + 1;   // bits [31, sh) of the k-th key are known
      __syncthreads();          // list_fill is zero for every warp
      int m = 0;
#pragma unroll
      for (int j = 0; j < kCache; ++j) {
        const bool valid = j < chunk && base + 32 * j < wend;
        m += valid && (sh >= 32 || (keys[j] >> sh) == (prefix >> sh));
      }
      int incl = m;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int x = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += x;
      }
      int wbase = 0;
      if (lane == 31 && incl) wbase = atomicAdd(&list_fill, incl);   // list order does not matter
      int pos = __shfl_sync(0xffffffffu, wbase, 31) + incl - m;
      if (m) {
#pragma unroll
        for (int j = 0; j < kCache; ++j) {
          const bool valid = j < chunk && base + 32 * j < wend;
          if (valid && (sh >= 32 || (keys[j] >> sh) == (prefix >> sh))) list[min(pos++, kThreads - 1)] = keys[j];
        }
      }
      __syncthreads();
      const uint32_t ck = (int)threadIdx.x < min(list_fill, kThreads) ? list[threadIdx.x] : 0u;
      for (; bit >= 0; --bit, par ^= 1) {
        const uint32_t cand = prefix | (1u << bit);
        const unsigned b = __ballot_sync(0xffffffffu, ck >= cand);
        if (lane == 0) wcnt[par][warp] = __popc(b);
        __syncthreads();
        if (above + __reduce_add_sync(0xffffffffu, wcnt[par][lane]) >= e) prefix = cand;
      }
    }
  } else {
    // 8 bits per pass from the top: after the loop `prefix` is the key of the e-th largest score
    uint32_t mask = 0;
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int i = lane; i < 256; i += 32) whist[warp][i] = 0;
      __syncwarp();
      // consecutive equal digits of a thread are added in one go (scores of one head share their top bits)
      int run_bin = -1, run_cnt = 0;
      for (int j = 0; j < chunk; ++j) {
        const int t = base + 32 * j;
        if (t >= wend) break;
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
        for (int i = 0; i < 8; ++i) cnt[i] = totals[8 * lane + i], mine += cnt[i];
        int incl = mine;   // matching keys in this lane's digits and in those of higher lanes
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
  }

  // ordered compaction.  First the per-warp totals of keys above and equal to the k-th ...
  int gt = 0, eq = 0;
  if (kCached) {
#pragma unroll
    for (int j = 0; j < kCache; ++j) gt += keys[j] > prefix, eq += keys[j] == prefix;
  } else {
    for (int j = 0; j < chunk; ++j) {
      const int t = base + 32 * j;
      if (t >= wend) break;
      const uint32_t key = key_of(sc[t]);
      gt += key > prefix, eq += key == prefix;
    }
  }
  gt = __reduce_add_sync(0xffffffffu, gt);
  eq = __reduce_add_sync(0xffffffffu, eq);
  __syncthreads();
  if (lane == 0) warp_gt[warp] = gt, warp_eq[warp] = eq;
  __syncthreads();
  if (warp == 0) {   // exclusive scan over the warps
    const int a = warp_gt[lane], b = warp_eq[lane];
    int ai = a, bi = b;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, ai, o), y = __shfl_up_sync(0xffffffffu, bi, o);
      if (lane >= o) ai += x, bi += y;
    }
    warp_gt[lane] = ai - a;
    warp_eq[lane] = bi - b;
    if (lane == 31) sh_want = e - ai;   // keys equal to the k-th that are kept: k minus all keys above it
  }
  __syncthreads();
  want = sh_want;
  // ... then, row by row of the warp's range, ballots give every kept position its rank
  int gt_run = warp_gt[warp], eq_run = warp_eq[warp];
  const unsigned lt = (1u << lane) - 1u;
  auto place_row = [&](uint32_t key, bool valid, int t) {
    const unsigned gm = __ballot_sync(0xffffffffu, valid && key > prefix);
    const unsigned em = __ballot_sync(0xffffffffu, valid && key == prefix);
    const int gt_before = gt_run + __popc(gm & lt), eq_before = eq_run + __popc(em & lt);
    if (valid) {
      if (key > prefix) out[gt_before + min(eq_before, want)] = t;
      else if (key == prefix && eq_before < want) out[gt_before + eq_before] = t;
    }
    gt_run += __popc(gm), eq_run += __popc(em);
  };
  if (kCached) {
#pragma unroll
    for (int j = 0; j < kCache; ++j) {
      const int t = base + 32 * j;
      place_row(keys[j], j < chunk && t < wend, t);
    }
  } else {
    for (int j = 0; j < chunk; ++j) {
      const int t = base + 32 * j;
      const bool valid = t < wend;
      place_row(valid ? key_of(sc[t]) : 0u, valid, t);
    }
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
