// Diagnostic of Prop. 4.1: the attention mass of every observation-window row that survives the selection,
//   kept[u,h,i] = sum_{t in S_g, t <= n+i} A^h[n+i, t],
// so that the discarded mass is m = 1 - kept.  The window rows stand in for decode queries: their softmax
// normalisers are already in the work space (the row statistics the scan's first pass leaves), so the kernel only
// has to visit the retained rows of K~: logits against the gathered keys, exp2 against the stored row
// log-sum-exp.  Reading K~ rather than K makes it a consumer check of the gather as well.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 128;
constexpr int kTileRows = 32;   // retained rows staged per step

template <bool BF16>
__device__ __forceinline__ float load_elem(const char* p, int64_t i) {
  if (BF16) return __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(p)[i] << 16);
  return reinterpret_cast<const float*>(p)[i];
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads) kept_mass_kernel(ckv_shape s, int RB, int hpb, int64_t unit_rows,
                                                             const char* __restrict__ q, const char* __restrict__ k_out,
                                                             const int32_t* __restrict__ indices,
                                                             const int32_t* __restrict__ budgets,
                                                             const int32_t* __restrict__ offsets,
                                                             const float2* __restrict__ stat_plain,
                                                             const float2* __restrict__ stat_tc,
                                                             const int* __restrict__ marker, float* __restrict__ kept) {
  __shared__ float tile[kTileRows][kHeadDim + 1];
  __shared__ int tpos[kTileRows];
  __shared__ float partial[kThreads];
  const int u = blockIdx.y, h = blockIdx.x;
  const int W = s.window, L = s.seq_len, n = L - W, H = s.n_q_heads, Hkv = s.n_kv_heads, G = H / Hkv, g = h / G;
  const int i = threadIdx.x % W, part = threadIdx.x / W, parts = kThreads / W;   // W <= 64: at least two parts
  const bool active = part < parts;
  // the row's log2-domain log-sum-exp, from whichever scan wrote this work space
  float lse;
  if ((*marker & 0xff) == 2) {
    const int rb = (h - g * G) / hpb, head0 = g * G + rb * hpb;
    const int64_t chunk = ((int64_t)u * Hkv + g) * RB + rb;
    lse = stat_tc[chunk * 128 + (h - head0) * W + i].y;
  } else {
    lse = stat_plain[((int64_t)u * H + h) * W + i].y;
  }
  float qv[kHeadDim];
  {
    const int64_t qo = (int64_t)u * s.q_stride_unit + (int64_t)h * s.q_stride_head + (int64_t)i * s.q_stride_row;
#pragma unroll
    for (int d = 0; d < kHeadDim; ++d) qv[d] = load_elem<BF16>(q, qo + d);
  }
  const int rows = budgets[(int64_t)u * Hkv + g];
  const int64_t base = (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g];
  float acc = 0.f;
  for (int r0 = 0; r0 < rows; r0 += kTileRows) {
    __syncthreads();
    for (int e = threadIdx.x; e < kTileRows * kHeadDim; e += kThreads) {
      const int r = e / kHeadDim, d = e - r * kHeadDim;
      tile[r][d] = r0 + r < rows ? load_elem<BF16>(k_out, (base + r0 + r) * kHeadDim + d) : 0.f;
    }
    if (threadIdx.x < kTileRows) tpos[threadIdx.x] = r0 + (int)threadIdx.x < rows ? indices[base + r0 + threadIdx.x] : L;
    __syncthreads();
    if (active) {
      for (int r = part; r < kTileRows; r += parts) {
        if (tpos[r] > n + i) continue;   // past the end, or a window key this row cannot see
        float dot = 0.f;
#pragma unroll
        for (int d = 0; d < kHeadDim; ++d) dot = fmaf(qv[d], tile[r][d], dot);
        acc += exp2f(dot * (kLog2e * 0.08838834764831845f) - lse);
      }
    }
  }
  partial[threadIdx.x] = active ? acc : 0.f;
  __syncthreads();
  if (threadIdx.x < W) {
    float tot = 0.f;
    for (int p = 0; p < parts; ++p) tot += partial[p * W + threadIdx.x];
    kept[((int64_t)u * H + h) * W + threadIdx.x] = tot;
  }
}

}  // namespace

cudaError_t launch_kept_mass(const ckv_shape& s, const ckv_params& p, const void* q, const void* k_out,
                             const int32_t* indices, const int32_t* budgets, const int32_t* offsets,
                             const void* stat_plain, const void* stat_tc, const int* marker, float* kept,
                             cudaStream_t st) {
  const int hpb = 128 / s.window < 1 ? 1 : 128 / s.window;
  const int G = s.n_q_heads / s.n_kv_heads;
  const int RB = (G + hpb - 1) / hpb;
  const int64_t unit_rows = (int64_t)s.n_kv_heads * (p.budget_per_head < s.seq_len ? p.budget_per_head : s.seq_len);
  dim3 grid(s.n_q_heads, s.n_units);
  if (s.dtype == CKV_BF16)
    kept_mass_kernel<true><<<grid, kThreads, 0, st>>>(s, RB, hpb, unit_rows, (const char*)q, (const char*)k_out, indices,
                                                      budgets, offsets, (const float2*)stat_plain,
                                                      (const float2*)stat_tc, marker, kept);
  else
    kept_mass_kernel<false><<<grid, kThreads, 0, st>>>(s, RB, hpb, unit_rows, (const char*)q, (const char*)k_out, indices,
                                                       budgets, offsets, (const float2*)stat_plain,
                                                       (const float2*)stat_tc, marker, kept);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
