// Token-subset gather / scatter (paper: token pruning keeps a subset of the video tokens; attention then
// runs over the kept tokens only).  dst[b,h,m,:] = src[b,h,idx[b,m],:] and the inverse.  Pure data
// movement: one 16-byte vector per thread and step, rows of d elements are contiguous, HBM-bound
// (2 * M * d * elem bytes per head).
#include "common.cuh"

namespace sva {

// SCATTER = false: dst row m <- src row idx[b][m];  SCATTER = true: dst row idx[b][m] <- src row m.
// An index outside [0, n_src_or_dst) is reported and its row skipped.
template <bool SCATTER>
__global__ void __launch_bounds__(256)
token_move_kernel(const uint8_t* __restrict__ src, Strides ss, uint8_t* __restrict__ dst, Strides sd,
                  const int32_t* __restrict__ idx, int H, int M, int n_full, int row_bytes, int elem_bytes,
                  int32_t* __restrict__ status) {
  const int vpr = row_bytes / 16;                       // 16-byte vectors per row
  const int bh = blockIdx.y, b = bh / H, h = bh % H;
  const long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int m = (int)(v / vpr), c = (int)(v % vpr);
  if (m >= M) return;
  const int t = __ldg(idx + (long long)b * M + m);
  if (t < 0 || t >= n_full) {
    if (c == 0 && status) atomicOr(status, SVA_DEV_BAD_INDEX);
    return;
  }
  const long long rs = SCATTER ? m : t, rd = SCATTER ? t : m;
  const uint4* s = reinterpret_cast<const uint4*>(src + ((long long)b * ss.b + (long long)h * ss.h + rs * ss.n) * elem_bytes) + c;
  uint4* d = reinterpret_cast<uint4*>(dst + ((long long)b * sd.b + (long long)h * sd.h + rd * sd.n) * elem_bytes) + c;
  *d = __ldg(s);
}

int launch_token_move(bool scatter, const void* src, const int64_t ss[3], void* dst, const int64_t sd[3],
                      const int32_t* idx, int B, int H, int M, int n_full, int d, int elem_bytes,
                      int32_t* status, cudaStream_t st) {
  const int row_bytes = d * elem_bytes;
  const long long vecs = (long long)M * (row_bytes / 16);
  dim3 grid((unsigned)((vecs + 255) / 256), (unsigned)(B * H));
  if (scatter)
    token_move_kernel<true><<<grid, 256, 0, st>>>((const uint8_t*)src, make_strides(ss), (uint8_t*)dst, make_strides(sd),
                                                  idx, H, M, n_full, row_bytes, elem_bytes, status);
  else
    token_move_kernel<false><<<grid, 256, 0, st>>>((const uint8_t*)src, make_strides(ss), (uint8_t*)dst, make_strides(sd),
                                                   idx, H, M, n_full, row_bytes, elem_bytes, status);
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

}  // namespace sva
