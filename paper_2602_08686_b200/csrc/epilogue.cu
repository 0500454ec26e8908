// Pooling, head-table weighting and group max (Eq. 4's L/W scale, Eq. 6 inside a GQA group), the
// unit's column mass and the per-CTA partial sums of its entropy (Eq. 7), in one pass over the
// per-head column sums.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 128;
constexpr int kPerThread = 4;                    // consecutive positions per thread
constexpr int kSpan = kThreads * kPerThread;     // positions per CTA
constexpr int kHeadBatch = 8;                    // heads staged in shared memory at a time
static_assert(kSpan == kEntSpan, "one entropy partial per CTA");

// Sum over the CTA's positions of -p ln p with p = mass / (W H); thread i holds positions 4 i .. 4 i + 3 and
// passes zero for those past the end.  Fixed order: the thread's four terms, a shuffle tree, the warps in
// index order.  Every thread must call; thread 0 gets the sum.
__device__ __forceinline__ double entropy_partial(const float (&mass)[kPerThread], double norm) {
  __shared__ double warp_sum[kThreads / 32];
  double acc = 0.0;
#pragma unroll
  for (int e = 0; e < kPerThread; ++e) {
    const double pt = (double)mass[e] * norm;
    if (pt > 0.0) acc -= pt * log(pt);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = acc;
  __syncthreads();
  double tot = 0.0;
  if (threadIdx.x == 0)
    for (int w = 0; w < kThreads / 32; ++w) tot += warp_sum[w];
  return tot;
}

// The same partials from a column mass that is already in memory (the stand-alone budget call).
__global__ void __launch_bounds__(kThreads) entropy_partials(ckv_shape s, const float* __restrict__ colmass,
                                                             double* __restrict__ ent_part,
                                                             int* __restrict__ done) {
  const int u = blockIdx.y, L = s.seq_len, tb = blockIdx.x * kSpan + threadIdx.x * kPerThread;
  float mass[kPerThread];
#pragma unroll
  for (int e = 0; e < kPerThread; ++e) mass[e] = tb + e < L ? colmass[(int64_t)u * L + tb + e] : 0.f;
  const double tot = entropy_partial(mass, 1.0 / ((double)s.window * (double)s.n_q_heads));
  if (threadIdx.x == 0) {
    ent_part[(int64_t)u * gridDim.x + blockIdx.x] = tot;
    if (blockIdx.x == 0) done[u] = 0;
  }
}

// One CTA owns kSpan consecutive positions t of one unit and walks over all query heads:
//   scores[u,g,t] = max_{h in g} head_w[h] * pool((L/W) c_h)[t]   for t < n  (pooling never looks past n)
//   colmass[u,t]  = sum_h c_h[t]                                    for t < L  (heads added in index order)
// R is the pooling radius (window 2R + 1); AVG counts positions outside the prefix as zeros and divides
// by the window size, MAX ignores them.
// GROUPED: csum holds one row per KV group that is already weighted, scaled and maximised over the
// group's heads (max pooling commutes with that for weights >= 0), and gmass the groups' column mass:
//   scores[u,g,t] = pool(csum[u,g])[t],   colmass[u,t] = sum_g gmass[u,g,t]   (groups in index order)
template <int R, bool AVG, bool GROUPED>
__global__ void __launch_bounds__(kThreads) pool_weight_max_mass(ckv_shape s, ckv_params p,
                                                                 const float* __restrict__ csum,
                                                                 const float* __restrict__ gmass,
                                                                 const float* __restrict__ head_w,
                                                                 float* __restrict__ scores,
                                                                 float* __restrict__ colmass,
                                                                 double* __restrict__ ent_part,
                                                                 int* __restrict__ done, int* __restrict__ marker,
                                                                 int marker_value) {
  pdl_launch_dependents();   // the counting kernel may be scheduled while this grid drains
  constexpr int kHalo = (R + 3) / 4 * 4;           // halo rounded up so that every thread's window is 16-byte aligned
  constexpr int kWidth = kSpan + 2 * kHalo;        // staged positions t0 - kHalo .. t0 + kSpan + kHalo - 1
  constexpr int kWin = kPerThread + 2 * kHalo;     // values a thread reads: c_h[tb - kHalo .. tb + 3 + kHalo]
  __shared__ __align__(16) float tile[kHeadBatch][kWidth];
  const int L = s.seq_len, n = L - s.window;
  const int H = GROUPED ? s.n_kv_heads : s.n_q_heads, G = GROUPED ? 1 : H / s.n_kv_heads;   // rows of csum
  const int u = blockIdx.y, t0 = blockIdx.x * kSpan, tb = t0 + threadIdx.x * kPerThread;
  const float scale = GROUPED ? 1.f : (float)L / (float)s.window;
  const float inv_size = 1.f / (float)(2 * R + 1);
  const float pad = AVG ? 0.f : -INFINITY;
  const float* hw = head_w + (int64_t)u * p.head_w_stride_unit;
  // a CTA whose staged range lies inside the prefix needs no range checks at all
  const bool interior = t0 - kHalo >= 0 && t0 + kSpan + kHalo <= n;
  float mass[kPerThread], best[kPerThread];
#pragma unroll
  for (int e = 0; e < kPerThread; ++e) mass[e] = 0.f, best[e] = -INFINITY;
  for (int h0 = 0; h0 < H; h0 += kHeadBatch) {
    const int nh = min(kHeadBatch, H - h0);
    __syncthreads();
    {
      // all loads of the batch first, then the stores: the loads are independent and overlap
      constexpr int kIters = (kWidth + kThreads - 1) / kThreads;
      float buf[kHeadBatch][kIters];
      float gm[GROUPED ? kHeadBatch : 1][kPerThread];
      if (GROUPED) {
#pragma unroll
        for (int hh = 0; hh < kHeadBatch; ++hh) {
          const float* m = gmass + ((int64_t)u * H + h0 + (hh < nh ? hh : 0)) * L;
#pragma unroll
          for (int e = 0; e < kPerThread; ++e) gm[hh][e] = (hh < nh && (interior || tb + e < L)) ? m[tb + e] : 0.f;
        }
      }
#pragma unroll
      for (int hh = 0; hh < kHeadBatch; ++hh) {
        const float* c = csum + ((int64_t)u * H + h0 + (hh < nh ? hh : 0)) * L;
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
          const int i = threadIdx.x + it * kThreads;
          const int tt = t0 - kHalo + i;
          buf[hh][it] = (hh < nh && i < kWidth && (interior || (tt >= 0 && tt < L))) ? c[tt] : 0.f;
        }
      }
#pragma unroll
      for (int hh = 0; hh < kHeadBatch; ++hh) {
#pragma unroll
        for (int it = 0; it < kIters; ++it) {
          const int i = threadIdx.x + it * kThreads;
          if (i < kWidth) tile[hh][i] = buf[hh][it];
        }
      }
      if (GROUPED) {
#pragma unroll
        for (int hh = 0; hh < kHeadBatch; ++hh)
#pragma unroll
          for (int e = 0; e < kPerThread; ++e) mass[e] += gm[hh][e];   // zero beyond the batch
      }
    }
    __syncthreads();
    for (int hh = 0; hh < nh; ++hh) {
      const int h = h0 + hh;
      float win[kWin];   // win[i] = c_h[tb - kHalo + i]
      const float4* src = reinterpret_cast<const float4*>(tile[hh] + threadIdx.x * kPerThread);
#pragma unroll
      for (int q4 = 0; q4 < kWin / 4; ++q4) {
        const float4 x = src[q4];
        win[4 * q4] = x.x, win[4 * q4 + 1] = x.y, win[4 * q4 + 2] = x.z, win[4 * q4 + 3] = x.w;
      }
      if (!GROUPED) {
#pragma unroll
        for (int e = 0; e < kPerThread; ++e)
          if (interior || tb + e < L) mass[e] += win[kHalo + e];
      }
      if (!interior) {   // the pooling only sees the prefix [0, n)
#pragma unroll
        for (int i = 0; i < kWin; ++i) {
          const int tt = tb - kHalo + i;
          if (tt < 0 || tt >= n) win[i] = pad;
        }
      }
      const float w = GROUPED ? 1.f : hw[h];
#pragma unroll
      for (int e = 0; e < kPerThread; ++e) {
        float v = win[kHalo + e - R];
#pragma unroll
        for (int i = 1; i <= 2 * R; ++i) v = AVG ? v + win[kHalo + e - R + i] : fmaxf(v, win[kHalo + e - R + i]);
        v = AVG ? v * scale * inv_size : v * scale;
        best[e] = fmaxf(best[e], w * v);
      }
      if ((h + 1) % G == 0) {  // last head of its KV group
        float* out = scores + ((int64_t)u * s.n_kv_heads + h / G) * n;
#pragma unroll
        for (int e = 0; e < kPerThread; ++e) {
          if (tb + e < n) out[tb + e] = best[e];
          best[e] = -INFINITY;
        }
      }
    }
  }
#pragma unroll
  for (int e = 0; e < kPerThread; ++e) {
    if (tb + e < L) colmass[(int64_t)u * L + tb + e] = mass[e];
    else mass[e] = 0.f;
  }
  const double tot = entropy_partial(mass, 1.0 / ((double)s.window * (double)s.n_q_heads));
  if (threadIdx.x == 0) {
    ent_part[(int64_t)u * gridDim.x + blockIdx.x] = tot;
    if (blockIdx.x == 0) done[u] = 0;
    if (blockIdx.x == 0 && u == 0) *marker = marker_value;
  }
}

template <int R>
void launch_r(bool avg, dim3 grid, cudaStream_t st, const ckv_shape& s, const ckv_params& p, const float* csum,
              const float* head_w, float* scores, float* colmass, double* ent, int* done, int* mk, int mv) {
  if (avg)
    pool_weight_max_mass<R, true, false><<<grid, kThreads, 0, st>>>(s, p, csum, nullptr, head_w, scores, colmass, ent, done, mk, mv);
  else
    pool_weight_max_mass<R, false, false><<<grid, kThreads, 0, st>>>(s, p, csum, nullptr, head_w, scores, colmass, ent, done, mk, mv);
}

template <int R>
void launch_g(dim3 grid, cudaStream_t st, const ckv_shape& s, const ckv_params& p, const float* zgrp,
              const float* mgrp, float* scores, float* colmass, double* ent, int* done, int* mk, int mv) {
  pool_weight_max_mass<R, false, true><<<grid, kThreads, 0, st>>>(s, p, zgrp, mgrp, nullptr, scores, colmass, ent, done, mk, mv);
}

}  // namespace

cudaError_t launch_entropy_partials(const ckv_shape& s, const float* colmass, void* ent_part, void* done,
                                    cudaStream_t st) {
  dim3 grid((s.seq_len + kSpan - 1) / kSpan, s.n_units);
  entropy_partials<<<grid, kThreads, 0, st>>>(s, colmass, (double*)ent_part, (int*)done);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_epilogue(const ckv_shape& s, const ckv_params& p, const float* csum, const float* head_w,
                            float* scores, float* colmass, void* ent_part, void* done, int* marker, int marker_value,
                            cudaStream_t st) {
  double* ent = (double*)ent_part;
  int* dn = (int*)done;
  dim3 grid((s.seq_len + kSpan - 1) / kSpan, s.n_units);
  const int r = (p.pool_kind == CKV_POOL_NONE) ? 0 : p.pool_size / 2;
  const bool avg = p.pool_kind == CKV_POOL_AVG && r > 0;
  switch (r) {
    case 0: launch_r<0>(false, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
    case 1: launch_r<1>(avg, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
    case 2: launch_r<2>(avg, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
    case 3: launch_r<3>(avg, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
    case 4: launch_r<4>(avg, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
    case 5: launch_r<5>(avg, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
    case 6: launch_r<6>(avg, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
    default: launch_r<7>(avg, grid, st, s, p, csum, head_w, scores, colmass, ent, dn, marker, marker_value); break;
  }
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_epilogue_grouped(const ckv_shape& s, const ckv_params& p, const float* zgrp, const float* mgrp,
                                    float* scores, float* colmass, void* ent_part, void* done, int* marker,
                                    int marker_value, cudaStream_t st) {
  double* ent = (double*)ent_part;
  int* dn = (int*)done;
  dim3 grid((s.seq_len + kSpan - 1) / kSpan, s.n_units);
  const int r = (p.pool_kind == CKV_POOL_NONE) ? 0 : p.pool_size / 2;
  switch (r) {
    case 0: launch_g<0>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
    case 1: launch_g<1>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
    case 2: launch_g<2>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
    case 3: launch_g<3>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
    case 4: launch_g<4>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
    case 5: launch_g<5>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
    case 6: launch_g<6>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
    default: launch_g<7>(grid, st, s, p, zgrp, mgrp, scores, colmass, ent, dn, marker, marker_value); break;
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
