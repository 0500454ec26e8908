// Plain (SIMT, fp32 FFMA) window-score kernels: the path for fp32 inputs and for shapes the
// tensor-core kernels do not take.  Two passes over K (Sec. 3 softmax; Eq. 4 window mass):
//   pass 1: per window row the maximum and the sum of exponentials of its logits, per key block;
//   combine: the per-block pairs are merged in block order into (max, max + log2 sum);
//   pass 2: the logits are recomputed and c_h[t] = sum_i 2^(x[i,t] - bias_i) is written.
// One thread owns one key; the W accumulators of the window rows live in registers.
#include <cuda_bf16.h>

#include "ckv_common.cuh"

namespace ckv {
namespace {

template <typename T>
struct Load8;  // eight consecutive elements of a K row as floats
template <>
struct Load8<__nv_bfloat16> {
  static __device__ __forceinline__ void run(const __nv_bfloat16* p, float (&o)[8]) {
    const uint4 raw = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      o[2 * j] = __uint_as_float(w[j] << 16);
      o[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
    }
  }
};
template <>
struct Load8<float> {
  static __device__ __forceinline__ void run(const float* p, float (&o)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    o[0] = a.x, o[1] = a.y, o[2] = a.z, o[3] = a.w, o[4] = b.x, o[5] = b.y, o[6] = b.z, o[7] = b.w;
  }
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// x[i] = (q[h,i] . k[g,t]) * log2(e)/sqrt(d) for the thread's key t, -inf where the causal mask
// hides the key or the key does not exist.
template <typename T, int WT>
__device__ __forceinline__ void logits_for_key(const ckv_shape& s, const T* __restrict__ k_row, bool key_valid,
                                               int t, const float* __restrict__ q_s, float (&x)[WT]) {
  const int W = s.window, n = s.seq_len - s.window;
#pragma unroll
  for (int i = 0; i < WT; ++i) x[i] = 0.f;
  if (key_valid) {
    for (int c8 = 0; c8 < kHeadDim / 8; ++c8) {
      float kv[8];
      Load8<T>::run(k_row + c8 * 8, kv);
#pragma unroll
      for (int i = 0; i < WT; ++i) {
        const float4 qa = *reinterpret_cast<const float4*>(q_s + i * kHeadDim + c8 * 8);
        const float4 qb = *reinterpret_cast<const float4*>(q_s + i * kHeadDim + c8 * 8 + 4);
        float a = x[i];
        a = fmaf(qa.x, kv[0], a), a = fmaf(qa.y, kv[1], a), a = fmaf(qa.z, kv[2], a), a = fmaf(qa.w, kv[3], a);
        a = fmaf(qb.x, kv[4], a), a = fmaf(qb.y, kv[5], a), a = fmaf(qb.z, kv[6], a), a = fmaf(qb.w, kv[7], a);
        x[i] = a;
      }
    }
  }
  const float scale = kLog2e * rsqrtf((float)kHeadDim);
#pragma unroll
  for (int i = 0; i < WT; ++i) {
    const bool vis = key_valid && i < W && t <= n + i;
    x[i] = vis ? x[i] * scale : -INFINITY;
  }
}

template <typename T, int WT>
__device__ __forceinline__ void stage_q(const ckv_shape& s, const T* __restrict__ q, int u, int h, float* q_s) {
  const T* qh = q + (int64_t)u * s.q_stride_unit + (int64_t)h * s.q_stride_head;
  for (int e = threadIdx.x; e < WT * kHeadDim; e += blockDim.x) {
    const int i = e / kHeadDim, c = e % kHeadDim;
    q_s[e] = i < s.window ? to_float(qh[(int64_t)i * s.q_stride_row + c]) : 0.f;
  }
  __syncthreads();
}

template <typename T, int WT>
__global__ void __launch_bounds__(kPlainKeysPerBlock) score_pass1_plain(ckv_shape s, const T* __restrict__ q,
                                                                        const T* __restrict__ k,
                                                                        float2* __restrict__ part, int nblk) {
  __shared__ __align__(16) float q_s[WT * kHeadDim];
  __shared__ float red[kPlainKeysPerBlock / 32][WT];
  __shared__ float row_max[WT];
  const int u = blockIdx.z, h = blockIdx.y, blk = blockIdx.x;
  const int g = h / (s.n_q_heads / s.n_kv_heads);
  stage_q<T, WT>(s, q, u, h, q_s);
  const int t = blk * kPlainKeysPerBlock + threadIdx.x;
  const bool valid = t < s.seq_len;
  const T* k_row = k + (int64_t)u * s.kv_stride_unit + (int64_t)g * s.kv_stride_head + (int64_t)t * s.kv_stride_tok;
  float x[WT];
  logits_for_key<T, WT>(s, k_row, valid, t, q_s, x);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // block maximum of every row
#pragma unroll
  for (int i = 0; i < WT; ++i) {
    float m = x[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp][i] = m;
  }
  __syncthreads();
  if (threadIdx.x < WT) {
    float m = red[0][threadIdx.x];
    for (int w = 1; w < kPlainKeysPerBlock / 32; ++w) m = fmaxf(m, red[w][threadIdx.x]);
    row_max[threadIdx.x] = m;
  }
  __syncthreads();
  // block sum of 2^(x - max); warps are added in a fixed order
#pragma unroll
  for (int i = 0; i < WT; ++i) {
    const float m = row_max[i];
    float p = (x[i] == -INFINITY) ? 0.f : exp2f(x[i] - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) p += __shfl_xor_sync(0xffffffffu, p, o);
    __syncwarp();
    if (lane == 0) red[warp][i] = p;
  }
  __syncthreads();
  if (threadIdx.x < s.window) {
    const int i = threadIdx.x;
    float l = 0.f;
    for (int w = 0; w < kPlainKeysPerBlock / 32; ++w) l += red[w][i];
    part[(((int64_t)u * s.n_q_heads + h) * s.window + i) * nblk + blk] = make_float2(row_max[i], l);
  }
}

// One thread per (unit, head, window row): merge the per-block pairs in block order.
__global__ void score_combine_plain(int rows, int nblk, const float2* __restrict__ part, float2* __restrict__ stat) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const float2* p = part + (int64_t)r * nblk;
  float m = -INFINITY;
  for (int b = 0; b < nblk; ++b) m = fmaxf(m, p[b].x);
  float l = 0.f;
  for (int b = 0; b < nblk; ++b)
    if (p[b].y > 0.f) l += p[b].y * exp2f(p[b].x - m);
  stat[r] = make_float2(m, m + log2f(l));
}

template <typename T, int WT>
__global__ void __launch_bounds__(kPlainKeysPerBlock) score_pass2_plain(ckv_shape s, const T* __restrict__ q,
                                                                        const T* __restrict__ k,
                                                                        const float2* __restrict__ stat,
                                                                        float* __restrict__ csum) {
  __shared__ __align__(16) float q_s[WT * kHeadDim];
  __shared__ float bias[WT];
  const int u = blockIdx.z, h = blockIdx.y, blk = blockIdx.x;
  const int g = h / (s.n_q_heads / s.n_kv_heads);
  if (threadIdx.x < WT)
    bias[threadIdx.x] =
        threadIdx.x < s.window ? stat[((int64_t)u * s.n_q_heads + h) * s.window + threadIdx.x].y : 0.f;
  stage_q<T, WT>(s, q, u, h, q_s);
  const int t = blk * kPlainKeysPerBlock + threadIdx.x;
  const bool valid = t < s.seq_len;
  const T* k_row = k + (int64_t)u * s.kv_stride_unit + (int64_t)g * s.kv_stride_head + (int64_t)t * s.kv_stride_tok;
  float x[WT];
  logits_for_key<T, WT>(s, k_row, valid, t, q_s, x);
  float c = 0.f;
#pragma unroll
  for (int i = 0; i < WT; ++i) c += (x[i] == -INFINITY) ? 0.f : exp2f(x[i] - bias[i]);
  if (valid) csum[((int64_t)u * s.n_q_heads + h) * s.seq_len + t] = c;
}

template <typename T, int WT>
cudaError_t run(const ckv_shape& s, const void* q, const void* k, float* csum, float2* part, float2* stat, int nblk,
                cudaStream_t st) {
  dim3 grid(nblk, s.n_q_heads, s.n_units);
  score_pass1_plain<T, WT><<<grid, kPlainKeysPerBlock, 0, st>>>(s, (const T*)q, (const T*)k, part, nblk);
  const int rows = s.n_units * s.n_q_heads * s.window;
  score_combine_plain<<<(rows + 127) / 128, 128, 0, st>>>(rows, nblk, part, stat);
  score_pass2_plain<T, WT><<<grid, kPlainKeysPerBlock, 0, st>>>(s, (const T*)q, (const T*)k, stat, csum);
  count_launch(3);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_score_plain(const ckv_shape& s, const void* q, const void* k, float* csum, float2* part,
                               float2* stat, int nblk, cudaStream_t st) {
  const bool bf = s.dtype == CKV_BF16;
  if (s.window <= 16) return bf ? run<__nv_bfloat16, 16>(s, q, k, csum, part, stat, nblk, st)
                                : run<float, 16>(s, q, k, csum, part, stat, nblk, st);
  if (s.window <= 32) return bf ? run<__nv_bfloat16, 32>(s, q, k, csum, part, stat, nblk, st)
                                : run<float, 32>(s, q, k, csum, part, stat, nblk, st);
  return bf ? run<__nv_bfloat16, 64>(s, q, k, csum, part, stat, nblk, st)
            : run<float, 64>(s, q, k, csum, part, stat, nblk, st);
}

}  // namespace ckv
