// Per-head exact Top-k (Eq. 8's Top-B branch): a most-significant-bit-first search finds the key of
// the k-th largest score, then one ordered compaction writes the kept positions in ascending order;
// equal scores are resolved toward the lowest index, and the observation window is appended.
// One CTA per (unit, KV head); integer work only, bit-exact and deterministic.
//
// The bit-sliced kernel: thread i of a CTA owns the 32 consecutive positions from 32 i, a CTA 32768
// positions, and prefixes of up to eight times that are spread over the CTAs of a thread-block
// cluster.  The scores are read coalesced, turned into ordered keys and staged in shared memory, from
// where every thread fetches its own 128-byte line; a 32 x 32 bit transpose in registers leaves plane
// b holding bit b of the thread's 32 keys.  A search step then costs a few logic
// operations and population counts per thread whatever the number of keys, so two bits are decided per
// CTA-wide reduction (16 reductions for the whole key).  The search ends with one mask of the keys above
// the k-th and one of the keys equal to it; their population counts, scanned over the threads in position
// order, place every kept position.
//
// Still longer prefixes use 8-bit digits with per-warp histograms and re-read the scores in every pass.
#include <cooperative_groups.h>

#include <algorithm>
#include <atomic>

#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kSlicedMax = kThreads * 32;   // positions the bit-sliced kernel holds

// Order-preserving map from float bits to unsigned: larger float <=> larger key.
__device__ __forceinline__ uint32_t key_of(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// In-place transpose of a 32 x 32 bit matrix held as 32 words (five rounds of masked block swaps).
// With word r read as row r and bit 31 as the leftmost column, afterwards a[r] bit c equals the
// former a[31 - c] bit (31 - r).
__device__ __forceinline__ void transpose32(uint32_t (&a)[32]) {
#pragma unroll
  for (int s = 0; s < 5; ++s) {
    const int j = 16 >> s;
    const uint32_t m = s == 0 ? 0x0000ffffu : s == 1 ? 0x00ff00ffu : s == 2 ? 0x0f0f0f0fu : s == 3 ? 0x33333333u
                                                                                                     : 0x55555555u;
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      if ((k & j) == 0) {
        const uint32_t t = (a[k] ^ (a[k + j] >> j)) & m;
        a[k] ^= t;
        a[k + j] ^= t << j;
      }
    }
  }
}

// 4-byte asynchronous copy into shared memory; src_bytes 0 writes zeros and reads nothing.
__device__ __forceinline__ void async_copy4(uint32_t* dst, const float* src, int src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src),
               "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void async_copy_wait() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// Exchange of a search step's counts between the CTAs of a cluster: every warp sends its two words to each
// CTA with one asynchronous store that also credits the receiver's transaction barrier, so a step costs
// one trip across the cluster instead of a store and a cluster-wide barrier.
__device__ __forceinline__ uint32_t cluster_address(const void* local, int cta) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"((uint32_t)__cvta_generic_to_shared(local)), "r"(cta));
  return r;
}
__device__ __forceinline__ void barrier_init(uint64_t* bar, int arrivals) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(arrivals) : "memory");
}
__device__ __forceinline__ void barrier_expect(uint64_t* bar, int bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void store_credit(uint32_t dst, uint64_t v, uint32_t bar) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];" ::"r"(dst), "l"(v), "r"(bar) : "memory");
}
__device__ __forceinline__ bool barrier_test(uint64_t* bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"((uint32_t)__cvta_generic_to_shared(bar)), "r"(parity)
      : "memory");
  return done != 0;
}
// Waits for the phase with the given parity, for limit_ns at most.
__device__ __forceinline__ bool barrier_wait_bounded(uint64_t* bar, uint32_t parity, unsigned long long limit_ns) {
  if (barrier_test(bar, parity)) return true;
  unsigned long long t0, t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (barrier_test(bar, parity)) return true;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    if (t - t0 > limit_ns) return false;
  }
}
constexpr int kSelectTimeoutCode = 51;   // status word: a cluster exchange of the selection gave up

// kCluster CTAs of one thread-block cluster share a head: CTA r holds the positions from r * kSlicedMax.
// Every warp then sends its counts to all CTAs of the cluster through distributed shared memory.  A CTA (cluster) takes the heads blockIdx.x / kCluster, + stride, ...;
// the scores of its next head stream into the staging area while it searches the current one.
template <int kCluster>
__global__ void __launch_bounds__(kThreads) select_sliced_kernel(ckv_shape s, int64_t unit_rows,
                                                                 const float* __restrict__ scores,
                                                                 const int32_t* __restrict__ budgets,
                                                                 const int32_t* __restrict__ offsets,
                                                                 int32_t* __restrict__ indices, int* __restrict__ status,
                                                                 unsigned long long wait_ns) {
  extern __shared__ __align__(16) uint32_t stage[];   // [warps in use][1024] score bits in position order
  __shared__ __align__(8) uint2 wcnt[2][kCluster][kWarps];
  __shared__ uint32_t wtot[kWarps];
  __shared__ uint32_t ctot[kCluster];
  __shared__ __align__(8) uint64_t xbar[2];   // one transaction barrier per buffer of wcnt
  __shared__ volatile int dead_s;             // an exchange timed out here or in another CTA of the cluster
  pdl_launch_dependents();
  if constexpr (kCluster > 1) {
    if (threadIdx.x == 0) {
      barrier_init(&xbar[0], 1), barrier_init(&xbar[1], 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      dead_s = 0;
    }
    cooperative_groups::this_cluster().sync();   // nobody sends before every barrier of the cluster exists
  }
  uint32_t phase = 0;   // bit b: parity of the phase xbar[b] is in
  pdl_wait();   // budgets, offsets and scores come from the kernels before
  const int Hkv = s.n_kv_heads, W = s.window, n = s.seq_len - W;
  const int n_heads = s.n_units * Hkv, stride = (int)gridDim.x / kCluster;
  const int rank = blockIdx.x % kCluster;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int cbase = rank * kSlicedMax;                      // first position of this CTA
  const int first = cbase + 32 * (int)threadIdx.x;          // first position of this thread
  const int wbase = warp * 1024;                            // first position of the warp inside the CTA
  const bool staged = cbase + wbase < n;                    // the warp holds positions of the prefix
  uint32_t* const ws = stage + wbase;
  // A CTA that gave up tells the others, and all CTAs of the cluster leave after the same cluster barrier:
  // none sends to a CTA that is gone.
  auto leave_dead = [&]() {
    async_copy_wait();
    if ((int)threadIdx.x < kCluster) *cooperative_groups::this_cluster().map_shared_rank(const_cast<int*>(&dead_s), threadIdx.x) = 1;
    cooperative_groups::this_cluster().sync();
  };
  // every warp copies its own 1024 scores: nothing but the warp reads them
  auto prefetch = [&](int head) {
    if (!staged) return;
    const float* sc = scores + (int64_t)head * n;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const int t = cbase + wbase + 32 * j + lane;
      async_copy4(ws + 32 * j + lane, t < n ? sc + t : sc, t < n ? 4 : 0);
    }
  };
  // positions of the thread that exist, in fetch order (bit k <-> position first + (k + 4 lane) % 32)
  const int rot = (4 * lane) & 31;
  const int have = min(max(n - first, 0), 32);
  const uint32_t valid_pos = have >= 32 ? 0xffffffffu : ((1u << have) - 1u);

  int head = blockIdx.x / kCluster;
  if (head < n_heads) prefetch(head);
  // the branches below are taken by all CTAs of a cluster alike
  for (; head < n_heads; head += stride) {
    const int u = head / Hkv, g = head - u * Hkv;
    const int e = budgets[(int64_t)u * Hkv + g] - W;
    int32_t* out = indices + (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g];

    // a[31 - k] = key of position first + (k + 4 * lane) % 32: the 16-byte pieces of the thread's line are
    // fetched in an order rotated by the lane so that a quarter warp touches every bank once
    uint32_t a[32];
    async_copy_wait();
    __syncwarp();
    if (staged) {
      const uint4* line = reinterpret_cast<const uint4*>(ws + 32 * lane);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const uint4 v = line[(q + lane) & 7];
        a[31 - 4 * q] = key_of(__uint_as_float(v.x)), a[30 - 4 * q] = key_of(__uint_as_float(v.y));
        a[29 - 4 * q] = key_of(__uint_as_float(v.z)), a[28 - 4 * q] = key_of(__uint_as_float(v.w));
      }
    } else {
#pragma unroll
      for (int k = 0; k < 32; ++k) a[k] = 0u;
    }
    __syncwarp();   // the warp has read its lines: the next head's scores may overwrite them
    if (head + stride < n_heads) prefetch(head + stride);

    if (rank == 0)
      for (int i = threadIdx.x; i < W; i += kThreads) out[e + i] = n + i;
    if (e <= 0) continue;
    if (e >= n) {
      for (int t = cbase + threadIdx.x; t < min(n, cbase + kSlicedMax); t += kThreads) out[t] = t;
      continue;
    }
    transpose32(a);   // a[31 - b] bit k = bit b of the k-th fetched key

    uint32_t alive = __funnelshift_r(valid_pos, valid_pos, rot);   // keys equal to the decided bits so far
    uint32_t gt = 0u;                                              // keys above the k-th
    int above = 0;                                                 // their number over the whole head
    int tied = n;                                                  // keys of the whole head still in `alive`
#pragma unroll
    for (int st = 0; st < 16; ++st) {
      const uint32_t p1 = a[2 * st], p0 = a[2 * st + 1];   // planes of bits 31 - 2 st and 30 - 2 st
      const uint32_t h = alive & p1, l = alive & ~p1;
      const uint32_t h1 = h & p0, l1 = l & p0;
      const uint32_t r1 = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(h1) | ((uint32_t)__popc(h) << 16));
      const uint32_t r2 = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(l1));
      // the other buffer is written in the next step, this one again only after that step's barrier
      if constexpr (kCluster == 1) {
        if (lane == 0) wcnt[st & 1][0][warp] = make_uint2(r1, r2);
        __syncthreads();
      } else {
        uint64_t* bar = &xbar[st & 1];
        if (threadIdx.x == 0) barrier_expect(bar, kCluster * kWarps * (int)sizeof(uint2));
        if (lane < kCluster)
          store_credit(cluster_address(&wcnt[st & 1][rank][warp], lane), (uint64_t)r1 | ((uint64_t)r2 << 32),
                       cluster_address(bar, lane));
        if (warp == 0 && !barrier_wait_bounded(bar, (phase >> (st & 1)) & 1u, wait_ns) && lane == 0) {
          dead_s = 1;
          atomicCAS(status, 0, kSelectTimeoutCode);
        }
        __syncthreads();   // warp 0 has seen every CTA's counts arrive
        if (dead_s) {
          leave_dead();
          return;
        }
        phase ^= 1u << (st & 1);
      }
      uint32_t wx = 0, wy = 0;   // lane l adds warp l of every CTA: both 16-bit fields stay below 2^14
#pragma unroll
      for (int c = 0; c < kCluster; ++c) {
        const uint2 w = wcnt[st & 1][c][lane];
        wx += w.x, wy += w.y;
      }
      int t11, t1x;
      if constexpr (kCluster == 1) {
        const uint32_t t1 = __reduce_add_sync(0xffffffffu, wx);
        t11 = (int)(t1 & 0xffffu), t1x = (int)(t1 >> 16);
      } else {
        t11 = (int)__reduce_add_sync(0xffffffffu, wx & 0xffffu), t1x = (int)__reduce_add_sync(0xffffffffu, wx >> 16);
      }
      const int t01 = (int)__reduce_add_sync(0xffffffffu, wy);
      if (above + t11 >= e) {               // digit 11
        alive = h1, tied = t11;
      } else if (above + t1x >= e) {        // digit 10
        gt |= h1, above += t11, alive = h & ~p0, tied = t1x - t11;
      } else if (above + t1x + t01 >= e) {  // digit 01
        gt |= h, above += t1x, alive = l1, tied = t01;
      } else {                              // digit 00
        gt |= h | l1, above += t1x + t01, alive = l & ~p0, tied -= t1x + t01;
      }
      // every key that still matches is kept: the lower bits decide nothing (the same test in every thread
      // of the cluster, so all leave together)
      if (above + tied == e) break;
    }
    // alive: keys equal to the k-th; the lowest (e - above) positions among them are kept
    const int want = e - above;
    const uint32_t gtp = __funnelshift_l(gt, gt, rot), eqp = __funnelshift_l(alive, alive, rot);   // position order
    const uint32_t mine = (uint32_t)__popc(gtp) | ((uint32_t)__popc(eqp) << 16);
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t x = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += x;
    }
    if (lane == 31) wtot[warp] = incl;
    __syncthreads();
    const uint32_t wt = wtot[lane];
    const uint32_t before = __reduce_add_sync(0xffffffffu, lane < warp ? wt : 0u) + incl - mine;
    int gt_before = (int)(before & 0xffffu), eq_before = (int)(before >> 16);
    if constexpr (kCluster > 1) {   // kept keys of the CTAs holding lower positions
      const uint32_t total = __reduce_add_sync(0xffffffffu, wt);
      if (warp == 0 && lane < kCluster) *cooperative_groups::this_cluster().map_shared_rank(&ctot[rank], lane) = total;
      cooperative_groups::this_cluster().sync();
      if (dead_s) {   // set by a CTA that gave up, before this barrier
        async_copy_wait();
        return;
      }
      for (int c = 0; c < rank; ++c) gt_before += (int)(ctot[c] & 0xffffu), eq_before += (int)(ctot[c] >> 16);
    }
    uint32_t m = gtp | eqp;
    while (m) {
      const int j = __ffs((int)m) - 1;
      const uint32_t bit = 1u << j;
      m &= m - 1u;
      const int gb = gt_before + __popc(gtp & (bit - 1u)), eb = eq_before + __popc(eqp & (bit - 1u));
      if (gtp & bit) out[gb + min(eb, want)] = first + j;
      else if (eb < want) out[gb + eb] = first + j;
    }
  }
}

__global__ void __launch_bounds__(kThreads) select_digit_kernel(ckv_shape s, int64_t unit_rows,
                                                                const float* __restrict__ scores,
                                                                const int32_t* __restrict__ budgets,
                                                                const int32_t* __restrict__ offsets,
                                                                int32_t* __restrict__ indices) {
  // Warp w owns the contiguous positions [w * 32 * chunk, (w + 1) * 32 * chunk) and lane l of it the
  // positions w * 32 * chunk + 32 j + l: every load is coalesced and a ballot per j gives the order
  // inside the warp's range.
  __shared__ int whist[kWarps][256];   // one histogram per warp
  __shared__ int totals[256];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_want;
  __shared__ int warp_gt[kWarps], warp_eq[kWarps];
  pdl_launch_dependents();
  pdl_wait();
  const int Hkv = s.n_kv_heads, W = s.window, n = s.seq_len - W;
  const int u = blockIdx.x / Hkv, g = blockIdx.x % Hkv;
  const int e = budgets[(int64_t)u * Hkv + g] - W;
  int32_t* out = indices + (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g];
  const float* sc = scores + ((int64_t)u * Hkv + g) * n;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  for (int i = threadIdx.x; i < W; i += kThreads) out[e + i] = n + i;
  if (e <= 0) return;
  if (e >= n) {
    for (int t = threadIdx.x; t < n; t += kThreads) out[t] = t;
    return;
  }

  const int chunk = (n + kThreads - 1) / kThreads;      // positions per thread
  const int base = warp * 32 * chunk + lane;            // position of (j = 0); (j) is base + 32 j
  const int wend = min((warp + 1) * 32 * chunk, n);     // end of the warp's range

  // 8 bits per pass from the top: after the loop `prefix` is the key of the e-th largest score
  uint32_t prefix = 0, mask = 0;
  int want = e;
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

  // ordered compaction.  First the per-warp totals of keys above and equal to the k-th ...
  int gt = 0, eq = 0;
  for (int j = 0; j < chunk; ++j) {
    const int t = base + 32 * j;
    if (t >= wend) break;
    const uint32_t key = key_of(sc[t]);
    gt += key > prefix, eq += key == prefix;
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
  for (int j = 0; j < chunk; ++j) {
    const int t = base + 32 * j;
    const bool valid = t < wend;
    const uint32_t key = valid ? key_of(sc[t]) : 0u;
    const unsigned gm = __ballot_sync(0xffffffffu, valid && key > prefix);
    const unsigned em = __ballot_sync(0xffffffffu, valid && key == prefix);
    const int gt_before = gt_run + __popc(gm & lt), eq_before = eq_run + __popc(em & lt);
    if (valid) {
      if (key > prefix) out[gt_before + min(eq_before, want)] = t;
      else if (key == prefix && eq_before < want) out[gt_before + eq_before] = t;
    }
    gt_run += __popc(gm), eq_run += __popc(em);
  }
}


template <int kCluster>
cudaError_t launch_sliced(const ckv_shape& s, int n, int64_t unit_rows, const float* scores, const int32_t* budgets,
                          const int32_t* offsets, int32_t* indices, int* status, cudaStream_t st) {
  const int per_cta = (n + kCluster - 1) / kCluster;   // staging covers the fullest CTA
  const size_t smem = (size_t)((std::min(per_cta, kSlicedMax) + 1023) / 1024) * 1024 * sizeof(uint32_t);
  cudaError_t e = cudaFuncSetAttribute(select_sliced_kernel<kCluster>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kSlicedMax * (int)sizeof(uint32_t));
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kCluster == 1 ? smem : kSlicedMax * sizeof(uint32_t);
  cfg.stream = st;
  cudaLaunchAttribute attr[2] = {};
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCluster, attr[0].val.clusterDim.y = 1, attr[0].val.clusterDim.z = 1;
  attr[1] = pdl_attribute();
  cfg.attrs = attr, cfg.numAttrs = 2;
  // as many CTAs (clusters) as the device holds at once; each loops over its share of the heads
  // one CTA of this kernel fills an SM: the answer depends on the device only, and is remembered per device
  static std::atomic<int> resident_of[kMaxDevices];
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  int resident = resident_of[dev].load(std::memory_order_relaxed);
  if (resident == 0) {
    int sms = 0, clusters = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    clusters = sms / kCluster;
    if (kCluster > 1) {
      cfg.gridDim = dim3((unsigned)(sms / kCluster * kCluster));
      int active = 0;
      if (cudaOccupancyMaxActiveClusters(&active, select_sliced_kernel<kCluster>, &cfg) == cudaSuccess && active > 0)
        clusters = active;
      else
        (void)cudaGetLastError();
    }
    resident = clusters > 0 ? clusters : 1;
    resident_of[dev].store(resident, std::memory_order_relaxed);
  }
  const int n_heads = s.n_units * s.n_kv_heads;
  cfg.gridDim = dim3((unsigned)(std::min(n_heads, resident) * kCluster));
  return cudaLaunchKernelEx(&cfg, select_sliced_kernel<kCluster>, s, unit_rows, scores, budgets, offsets, indices, status,
                            wait_limit_ns());
}

}  // namespace

cudaError_t launch_select(const ckv_shape& s, const ckv_params& p, const float* scores, const int32_t* budgets,
                          const int32_t* offsets, int32_t* indices, int* status, cudaStream_t st) {
  const int n = s.seq_len - s.window;
  // unit u's indices start at u * unit_rows; its heads' budgets fill that exactly unless the selection is elastic
  const int64_t unit_rows = (int64_t)s.n_kv_heads * (p.budget_per_head < s.seq_len ? p.budget_per_head : s.seq_len);
  cudaError_t e;
  if (n <= kSlicedMax) e = launch_sliced<1>(s, n, unit_rows, scores, budgets, offsets, indices, status, st);
  else if (n <= 2 * kSlicedMax) e = launch_sliced<2>(s, n, unit_rows, scores, budgets, offsets, indices, status, st);
  else if (n <= 4 * kSlicedMax) e = launch_sliced<4>(s, n, unit_rows, scores, budgets, offsets, indices, status, st);
  else if (n <= 8 * kSlicedMax) e = launch_sliced<8>(s, n, unit_rows, scores, budgets, offsets, indices, status, st);
  else {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(s.n_units * s.n_kv_heads), cfg.blockDim = dim3(kThreads), cfg.stream = st;
    cudaLaunchAttribute attr = pdl_attribute();
    cfg.attrs = &attr, cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, select_digit_kernel, s, unit_rows, scores, budgets, offsets, indices);
  }
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ckv
