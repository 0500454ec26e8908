// Value-norm ratio of the stabilised utility (Eq. 4's rho; Alg. 1 (B)): rho[t] = |v_t|_2 / (mean_k |v_k|_2 + eps)
// per unit and KV head.  Two kernels: one streams V once (16-byte loads, 16 threads per bf16 row) and leaves
// the row norms and per-block sums of them; the other adds the block sums in a fixed order, divides, and
// optionally multiplies the prefix scores by the ratio (it is shared by the query heads of a KV group and
// non-negative, so it commutes with Eq. 6's maximum over the group).
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerBlock = kVnormRows;       // rows per CTA of the first kernel
constexpr int kRowsPerPass = kThreads / 16;     // 16 threads share a row
constexpr int kFinishSpan = 1024;               // positions per CTA of the second kernel

__device__ __forceinline__ float sumsq_bf16x8(uint4 x) {
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xffff0000u);
    s = fmaf(lo, lo, s);
    s = fmaf(hi, hi, s);
  }
  return s;
}
__device__ __forceinline__ float sumsq_f32x4(uint4 x) {
  const float a = __uint_as_float(x.x), b = __uint_as_float(x.y), c = __uint_as_float(x.z), d = __uint_as_float(x.w);
  return fmaf(a, a, fmaf(b, b, fmaf(c, c, d * d)));
}

// r[u,g,t] = |v[u,g,t,:]|_2;  part[u,g,blk] = sum of the block's norms (rows in index order per 16-row pass,
// passes in order: a fixed association)
template <bool BF16>
__global__ void __launch_bounds__(kThreads) vnorm_rows(ckv_shape s, const char* __restrict__ v, float* __restrict__ r,
                                                       float* __restrict__ part, int nblk) {
  __shared__ float lane_sum[kRowsPerPass];
  const int u = blockIdx.z, g = blockIdx.y, L = s.seq_len;
  const int piece = threadIdx.x & 15, rowlane = threadIdx.x >> 4;
  const int64_t esz = BF16 ? 2 : 4;
  const char* base = v + ((int64_t)u * s.kv_stride_unit + (int64_t)g * s.kv_stride_head) * esz;
  float* out = r + ((int64_t)u * s.n_kv_heads + g) * (int64_t)L;
  float acc = 0.f;
  constexpr int kPasses = kRowsPerBlock / kRowsPerPass, kBatch = 8;   // loads of kBatch rows in flight per thread
#pragma unroll 1
  for (int it0 = 0; it0 < kPasses; it0 += kBatch) {
    uint4 x[kBatch][BF16 ? 1 : 2];
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int t = blockIdx.x * kRowsPerBlock + (it0 + i) * kRowsPerPass + rowlane;
      const uint4* row = reinterpret_cast<const uint4*>(base + (int64_t)min(t, L - 1) * s.kv_stride_tok * esz);
      x[i][0] = __ldg(row + piece);
      if (!BF16) x[i][1] = __ldg(row + piece + 16);
    }
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int t = blockIdx.x * kRowsPerBlock + (it0 + i) * kRowsPerPass + rowlane;
      float ss = BF16 ? sumsq_bf16x8(x[i][0]) : sumsq_f32x4(x[i][0]) + sumsq_f32x4(x[i][BF16 ? 0 : 1]);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      if (piece == 0 && t < L) {
        const float nrm = sqrtf(ss);
        out[t] = nrm;
        acc += nrm;
      }
    }
  }
  if (piece == 0) lane_sum[rowlane] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float tot = 0.f;
    for (int i = 0; i < kRowsPerPass; ++i) tot += lane_sum[i];
    part[((int64_t)u * s.n_kv_heads + g) * nblk + blockIdx.x] = tot;
  }
}

// rho = r / (mean + eps) in place; scores[u,g,t] *= rho[u,g,t] for the prefix when scores is given
__global__ void __launch_bounds__(kThreads) vnorm_finish(ckv_shape s, float eps, float* __restrict__ r,
                                                         const float* __restrict__ part, int nblk,
                                                         float* __restrict__ scores) {
  __shared__ double red[kThreads];
  const int u = blockIdx.z, g = blockIdx.y, L = s.seq_len, n = L - s.window;
  const int64_t ug = (int64_t)u * s.n_kv_heads + g;
  double a = 0.0;
  for (int i = threadIdx.x; i < nblk; i += kThreads) a += (double)part[ug * nblk + i];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int o = kThreads / 2; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  const float denom = (float)(red[0] / (double)L + (double)eps);
#pragma unroll
  for (int k = 0; k < kFinishSpan / kThreads; ++k) {
    const int t = blockIdx.x * kFinishSpan + k * kThreads + threadIdx.x;
    if (t < L) {
      const float rho = r[ug * L + t] / denom;
      r[ug * L + t] = rho;
      if (scores && t < n) scores[ug * n + t] *= rho;
    }
  }
}

}  // namespace

cudaError_t launch_vnorm_rows(const ckv_shape& s, const void* v, float* rho, float* part, cudaStream_t st) {
  const int nblk = (s.seq_len + kRowsPerBlock - 1) / kRowsPerBlock;
  dim3 grid(nblk, s.n_kv_heads, s.n_units);
  if (s.dtype == CKV_BF16) vnorm_rows<true><<<grid, kThreads, 0, st>>>(s, (const char*)v, rho, part, nblk);
  else vnorm_rows<false><<<grid, kThreads, 0, st>>>(s, (const char*)v, rho, part, nblk);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_vnorm_finish(const ckv_shape& s, float eps, float* rho, const float* part, float* scores,
                                cudaStream_t st) {
  const int nblk = (s.seq_len + kRowsPerBlock - 1) / kRowsPerBlock;
  dim3 grid((s.seq_len + kFinishSpan - 1) / kFinishSpan, s.n_kv_heads, s.n_units);
  vnorm_finish<<<grid, kThreads, 0, st>>>(s, eps, rho, part, nblk, scores);
  count_launch();
  return cudaGetLastError();
}

}  // namespace ckv
