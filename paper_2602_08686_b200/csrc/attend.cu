// Decode-side check of the compressed cache (the setting of Prop. 4.1): softmax attention of a few decode queries
// per query head over either all L rows of K, V or the rows the retention pass gathered.  Not part of the retention
// pass; a diagnostic that consumes its output the way a decoder would.  Plain fp32 SIMT code: one CTA per (unit,
// KV head, slice of the rows), the group's queries (at most 32 rows: lane = row) against tiles of 64 keys staged
// in shared memory as fp32, an online softmax per row, partial results per slice merged by a second kernel.
#include "ckv_common.cuh"

namespace ckv {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTileKeys = 64;
constexpr int kKeysPerWarp = kTileKeys / kWarps;     // 8
constexpr int kDimsPerWarp = kHeadDim / kWarps;      // 16
constexpr int kPitch = kHeadDim + 4;                 // row pitch of the Q and K tiles: lanes hit different banks
constexpr float kNegBig = -1.0e30f;

struct AttendSmem {
  float q[kAttendMaxRows][kPitch];
  float k[kTileKeys][kPitch];
  float v[kTileKeys][kHeadDim];
  float p[kAttendMaxRows][kTileKeys + 1];
  float red[2][kAttendMaxRows][kWarps];
};

template <bool BF16>
__device__ __forceinline__ void load_row_piece(const char* base, int64_t elem, float* dst) {
  // eight consecutive elements (bf16) or four (fp32) from a 16-byte aligned address
  const uint4 x = *reinterpret_cast<const uint4*>(base + elem * (BF16 ? 2 : 4));
  const uint32_t w[4] = {x.x, x.y, x.z, x.w};
  if (BF16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      dst[2 * i] = __uint_as_float(w[i] << 16);
      dst[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) dst[i] = __uint_as_float(w[i]);
  }
}

// part_ml [Nu,Hkv,S,32] (running max, sum) in the base-2 domain; part_o [Nu,Hkv,S,32,128]
template <bool BF16>
__global__ void __launch_bounds__(kThreads) attend_partial(ckv_shape s, int n_dec, int S, int compressed,
                                                           int64_t unit_rows, const char* __restrict__ q,
                                                           const char* __restrict__ k, const char* __restrict__ v,
                                                           const int32_t* __restrict__ budgets,
                                                           const int32_t* __restrict__ offsets,
                                                           float2* __restrict__ part_ml, float* __restrict__ part_o) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  AttendSmem& sm = *reinterpret_cast<AttendSmem*>(smem_raw);
  const int sl = blockIdx.x, g = blockIdx.y, u = blockIdx.z;
  const int H = s.n_q_heads, Hkv = s.n_kv_heads, G = H / Hkv, L = s.seq_len, R = G * n_dec;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kVec = BF16 ? 8 : 4;   // elements per 16-byte piece
  // the rows this CTA attends over
  const int rows = compressed ? budgets[(int64_t)u * Hkv + g] : L;
  const int64_t row0 = compressed ? (int64_t)u * unit_rows + offsets[(int64_t)u * (Hkv + 1) + g] : 0;
  const int64_t tok_stride = compressed ? kHeadDim : s.kv_stride_tok;
  const int64_t base = compressed ? row0 * kHeadDim : (int64_t)u * s.kv_stride_unit + (int64_t)g * s.kv_stride_head;
  const int per = ((rows + S - 1) / S + kTileKeys - 1) / kTileKeys * kTileKeys;
  const int t_begin = min(sl * per, rows), t_end = min(t_begin + per, rows);
  // the group's query rows: row r = (head in group) * n_dec + query
  for (int e = threadIdx.x; e < kAttendMaxRows * (kHeadDim / kVec); e += kThreads) {
    const int r = e / (kHeadDim / kVec), c = e - r * (kHeadDim / kVec);
    float x[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (r < R) load_row_piece<BF16>(q, ((((int64_t)u * H + g * G + r / n_dec) * n_dec + r % n_dec) * kHeadDim) + c * kVec, x);
#pragma unroll
    for (int i = 0; i < kVec; ++i) sm.q[r][c * kVec + i] = x[i];
  }
  float m_run = kNegBig, l_run = 0.f;   // replicated in every warp for row = lane
  float acc[kDimsPerWarp];
#pragma unroll
  for (int i = 0; i < kDimsPerWarp; ++i) acc[i] = 0.f;
  const float scale = kLog2e * 0.08838834764831845f;   // log2(e) / sqrt(128)
  for (int t0 = t_begin; t0 < t_end; t0 += kTileKeys) {
    __syncthreads();   // the previous tile's readers are done (and the queries are in place)
    for (int e = threadIdx.x; e < kTileKeys * (kHeadDim / kVec); e += kThreads) {
      const int j = e / (kHeadDim / kVec), c = e - j * (kHeadDim / kVec);
      float xk[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, xv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (t0 + j < t_end) {
        const int64_t off = base + (int64_t)(t0 + j) * tok_stride + c * kVec;
        load_row_piece<BF16>(k, off, xk);
        load_row_piece<BF16>(v, off, xv);
      }
#pragma unroll
      for (int i = 0; i < kVec; ++i) sm.k[j][c * kVec + i] = xk[i], sm.v[j][c * kVec + i] = xv[i];
    }
    __syncthreads();
    // logits of row `lane` against this warp's eight keys
    float x[kKeysPerWarp];
#pragma unroll
    for (int jj = 0; jj < kKeysPerWarp; ++jj) x[jj] = 0.f;
#pragma unroll 4
    for (int d4 = 0; d4 < kHeadDim / 4; ++d4) {
      const float4 qv = *reinterpret_cast<const float4*>(&sm.q[lane][4 * d4]);
#pragma unroll
      for (int jj = 0; jj < kKeysPerWarp; ++jj) {
        const float4 kv = *reinterpret_cast<const float4*>(&sm.k[warp * kKeysPerWarp + jj][4 * d4]);
        x[jj] = fmaf(qv.x, kv.x, fmaf(qv.y, kv.y, fmaf(qv.z, kv.z, fmaf(qv.w, kv.w, x[jj]))));
      }
    }
    float mx = kNegBig;
#pragma unroll
    for (int jj = 0; jj < kKeysPerWarp; ++jj) {
      x[jj] = t0 + warp * kKeysPerWarp + jj < t_end ? x[jj] * scale : kNegBig;
      mx = fmaxf(mx, x[jj]);
    }
    sm.red[0][lane][warp] = mx;
    __syncthreads();
    float m_new = m_run;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) m_new = fmaxf(m_new, sm.red[0][lane][w]);
    float ps = 0.f;
#pragma unroll
    for (int jj = 0; jj < kKeysPerWarp; ++jj) {
      const float pj = x[jj] > 0.5f * kNegBig ? exp2f(x[jj] - m_new) : 0.f;
      sm.p[lane][warp * kKeysPerWarp + jj] = pj;
      ps += pj;
    }
    sm.red[1][lane][warp] = ps;
    __syncthreads();
    const float rescale = exp2f(m_run - m_new);   // 0 while nothing has been seen
    float tile_sum = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) tile_sum += sm.red[1][lane][w];
    l_run = l_run * rescale + tile_sum;
    m_run = m_new;
    // out[row][this warp's 16 dims] += p . v
#pragma unroll
    for (int i = 0; i < kDimsPerWarp; ++i) acc[i] *= rescale;
#pragma unroll 4
    for (int j = 0; j < kTileKeys; ++j) {
      const float pj = sm.p[lane][j];
#pragma unroll
      for (int i4 = 0; i4 < kDimsPerWarp / 4; ++i4) {
        const float4 vv = *reinterpret_cast<const float4*>(&sm.v[j][warp * kDimsPerWarp + 4 * i4]);
        acc[4 * i4] = fmaf(pj, vv.x, acc[4 * i4]);
        acc[4 * i4 + 1] = fmaf(pj, vv.y, acc[4 * i4 + 1]);
        acc[4 * i4 + 2] = fmaf(pj, vv.z, acc[4 * i4 + 2]);
        acc[4 * i4 + 3] = fmaf(pj, vv.w, acc[4 * i4 + 3]);
      }
    }
  }
  const int64_t slot = (((int64_t)u * Hkv + g) * S + sl) * kAttendMaxRows + lane;
  if (warp == 0) part_ml[slot] = make_float2(m_run, l_run);
#pragma unroll
  for (int i = 0; i < kDimsPerWarp; ++i) part_o[slot * kHeadDim + warp * kDimsPerWarp + i] = acc[i];
}

// out[u,h,j,:] and lse[u,h,j] (natural log) from the slices' partial results, slices in index order
__global__ void __launch_bounds__(kHeadDim) attend_merge(ckv_shape s, int n_dec, int S, const float2* __restrict__ part_ml,
                                                         const float* __restrict__ part_o, float* __restrict__ out,
                                                         float* __restrict__ lse) {
  const int r = blockIdx.x, g = blockIdx.y, u = blockIdx.z;
  const int H = s.n_q_heads, Hkv = s.n_kv_heads, G = H / Hkv;
  const int64_t first = ((int64_t)u * Hkv + g) * S * kAttendMaxRows + r;
  float M = kNegBig;
  for (int sl = 0; sl < S; ++sl) M = fmaxf(M, part_ml[first + (int64_t)sl * kAttendMaxRows].x);
  float Lsum = 0.f, o = 0.f;
  for (int sl = 0; sl < S; ++sl) {
    const float2 ml = part_ml[first + (int64_t)sl * kAttendMaxRows];
    const float w = ml.y > 0.f ? exp2f(ml.x - M) : 0.f;
    Lsum += ml.y * w;
    o += part_o[(first + (int64_t)sl * kAttendMaxRows) * kHeadDim + threadIdx.x] * w;
  }
  const int64_t row = ((int64_t)u * H + g * G + r / n_dec) * n_dec + r % n_dec;
  out[row * kHeadDim + threadIdx.x] = o / Lsum;
  if (threadIdx.x == 0) lse[row] = (M + log2f(Lsum)) * 0.6931471805599453f;
}

}  // namespace

int attend_slices(const ckv_shape& s) {
  const int64_t heads = (int64_t)s.n_units * s.n_kv_heads;
  const int64_t want = (4 * 148 + heads - 1) / heads;
  return (int)(want < 1 ? 1 : (want > 16 ? 16 : want));
}

cudaError_t launch_attend(const ckv_shape& s, const ckv_params& p, const void* q_dec, int n_dec, const void* k,
                          const void* v, int compressed, const int32_t* budgets, const int32_t* offsets, float* out,
                          float* lse, void* part_ml, void* part_o, cudaStream_t st) {
  const int S = attend_slices(s);
  const int G = s.n_q_heads / s.n_kv_heads;
  const int64_t unit_rows = (int64_t)s.n_kv_heads * (p.budget_per_head < s.seq_len ? p.budget_per_head : s.seq_len);
  dim3 grid(S, s.n_kv_heads, s.n_units);
  cudaError_t e;
  if (s.dtype == CKV_BF16) {
    e = cudaFuncSetAttribute(attend_partial<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttendSmem));
    if (e != cudaSuccess) return e;
    attend_partial<true><<<grid, kThreads, sizeof(AttendSmem), st>>>(
        s, n_dec, S, compressed, unit_rows, (const char*)q_dec, (const char*)k, (const char*)v, budgets, offsets,
        (float2*)part_ml, (float*)part_o);
  } else {
    e = cudaFuncSetAttribute(attend_partial<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(AttendSmem));
    if (e != cudaSuccess) return e;
    attend_partial<false><<<grid, kThreads, sizeof(AttendSmem), st>>>(
        s, n_dec, S, compressed, unit_rows, (const char*)q_dec, (const char*)k, (const char*)v, budgets, offsets,
        (float2*)part_ml, (float*)part_o);
  }
  attend_merge<<<dim3(G * n_dec, s.n_kv_heads, s.n_units), kHeadDim, 0, st>>>(s, n_dec, S, (const float2*)part_ml,
                                                                              (const float*)part_o, out, lse);
  count_launch(2);
  return cudaGetLastError();
}

}  // namespace ckv
