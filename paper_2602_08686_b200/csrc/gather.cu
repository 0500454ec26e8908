// Gather of the retained K/V rows (K~ = K[S], V~ = V[S]; Sec. 3, Alg. 1 (D)): bit copies in
// 16-byte vectors; consecutive threads move consecutive 16-byte pieces of one row, so both the
// reads (one full row = 256 or 512 bytes) and the writes are fully coalesced.
#include "ckv_common.cuh"

namespace ckv {
namespace {

__global__ void __launch_bounds__(256) gather_kernel(ckv_shape s, int rows_per_head, int vec_per_row,
                                                     const uint4* __restrict__ k, const uint4* __restrict__ v,
                                                     const int32_t* __restrict__ indices,
                                                     const int32_t* __restrict__ offsets, uint4* __restrict__ k_out,
                                                     uint4* __restrict__ v_out) {
  pdl_wait();   // indices and offsets come from the kernels before
  const int Hkv = s.n_kv_heads;
  const int64_t rows_per_unit = (int64_t)Hkv * rows_per_head;
  const int64_t total = (int64_t)s.n_units * rows_per_unit * vec_per_row;
  const int elems_per_vec = (s.dtype == CKV_BF16) ? 8 : 4;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / vec_per_row;
    const int piece = (int)(i - row * vec_per_row);
    const int u = (int)(row / rows_per_unit);
    const int r = (int)(row - (int64_t)u * rows_per_unit);
    const int32_t* off = offsets + (int64_t)u * (Hkv + 1);
    if (r >= off[Hkv]) continue;   // an elastic selection keeps fewer rows than the unit's share of the output
    int g = 0;
    while (g + 1 < Hkv && r >= off[g + 1]) ++g;
    const int t = indices[row];
    if ((unsigned)t >= (unsigned)s.seq_len) {  // never produced by ckv_select; guards against foreign index buffers
      k_out[i] = make_uint4(0u, 0u, 0u, 0u);
      v_out[i] = make_uint4(0u, 0u, 0u, 0u);
      continue;
    }
    const int64_t src =
        ((int64_t)u * s.kv_stride_unit + (int64_t)g * s.kv_stride_head + (int64_t)t * s.kv_stride_tok) / elems_per_vec +
        piece;
    k_out[i] = k[src];
    v_out[i] = v[src];
  }
}

}  // namespace

cudaError_t launch_gather(const ckv_shape& s, const ckv_params& p, const void* k, const void* v,
                          const int32_t* indices, const int32_t* offsets, void* k_out, void* v_out,
                          cudaStream_t st) {
  const int rows_per_head = p.budget_per_head < s.seq_len ? p.budget_per_head : s.seq_len;
  const int esz = s.dtype == CKV_BF16 ? 2 : 4;
  const int vec_per_row = kHeadDim * esz / 16;
  const int64_t total = (int64_t)s.n_units * s.n_kv_heads * rows_per_head * vec_per_row;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (blocks < 1) blocks = 1;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)blocks), cfg.blockDim = dim3(256), cfg.stream = st;
  cudaLaunchAttribute attr = pdl_attribute();
  cfg.attrs = &attr, cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, gather_kernel, s, rows_per_head, vec_per_row, (const uint4*)k,
                                           (const uint4*)v, indices, offsets, (uint4*)k_out, (uint4*)v_out);
  count_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace ckv
