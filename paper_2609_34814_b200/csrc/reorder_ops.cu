// Drop-in reorder operators of the paper's deployment mode (Section 5): gather the query
// blocks (and the mask rows) into the planned order before an unmodified attention backend,
// and scatter the output blocks back afterwards.  waveal_bsattn_fwd does not need them (it
// walks the order as an index list); they exist so that the plan can drive another backend,
// and so that the cost of the two extra passes the paper pays can be measured.
// Both are pure HBM copies: one CTA moves one block of `block` tokens with 16-byte accesses.
#include "host_common.h"

namespace {

// dst block (h, p) <- src block (h, order[h][p])   (gather)   or
// dst block (h, order[h][p]) <- src block (h, p)   (scatter)
template <bool SCATTER>
__global__ void __launch_bounds__(256) k_move_blocks(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                      const int* __restrict__ order, int n_blocks,
                                                      int vec_per_token, int block_tokens,
                                                      long long src_stride_h, long long src_stride_t,
                                                      long long dst_stride_h, long long dst_stride_t) {
  const int p = blockIdx.x, h = blockIdx.y;
  int r = order[(size_t)h * n_blocks + p];
  if (r < 0 || r >= n_blocks) return;                       // malformed order: touch nothing
  const int sb = SCATTER ? p : r, db = SCATTER ? r : p;
  const uint4* s = src + (size_t)h * src_stride_h + (size_t)sb * block_tokens * src_stride_t;
  uint4* d = dst + (size_t)h * dst_stride_h + (size_t)db * block_tokens * dst_stride_t;
  const int total = block_tokens * vec_per_token;
  for (int i = threadIdx.x; i < total; i += blockDim.x) {
    const int t = i / vec_per_token, v = i - t * vec_per_token;
    d[(size_t)t * dst_stride_t + v] = __ldg(&s[(size_t)t * src_stride_t + v]);
  }
}

waveal_status move_blocks(bool scatter, int32_t heads, int32_t n_blocks, int32_t block, int32_t row_bytes,
                          const void* src, const int64_t* src_stride, void* dst, const int64_t* dst_stride,
                          const int32_t* row_order, cudaStream_t st) {
  if (heads <= 0 || n_blocks <= 0 || block <= 0 || row_bytes <= 0)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "heads, n_blocks, block and row_bytes must be positive");
  if (!src || !dst || !row_order || !src_stride || !dst_stride)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "src, dst, strides and row_order are required");
  if (row_bytes % 16 || src_stride[0] % 16 || src_stride[1] % 16 || dst_stride[0] % 16 || dst_stride[1] % 16)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "row_bytes and byte strides must be multiples of 16");
  if (src_stride[1] < row_bytes || dst_stride[1] < row_bytes)
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "token strides must be at least row_bytes");
  if (!waveal::aligned(src, 16) || !waveal::aligned(dst, 16))
    return waveal::fail(WAVEAL_ERR_INVALID_ARG, "src and dst must be 16-byte aligned");
  if (heads > 65535) return waveal::fail(WAVEAL_ERR_UNSUPPORTED, "more than 65535 heads");
  dim3 grid((unsigned)n_blocks, (unsigned)heads);
  const uint4* s = static_cast<const uint4*>(src);
  uint4* d = static_cast<uint4*>(dst);
  if (scatter)
    k_move_blocks<true><<<grid, 256, 0, st>>>(s, d, row_order, n_blocks, row_bytes / 16, block, src_stride[0] / 16,
                                              src_stride[1] / 16, dst_stride[0] / 16, dst_stride[1] / 16);
  else
    k_move_blocks<false><<<grid, 256, 0, st>>>(s, d, row_order, n_blocks, row_bytes / 16, block, src_stride[0] / 16,
                                               src_stride[1] / 16, dst_stride[0] / 16, dst_stride[1] / 16);
  WAVEAL_CUDA_OK(cudaGetLastError());
  waveal::launch_counter() = 1;
  return WAVEAL_OK;
}

}  // namespace

extern "C" waveal_status waveal_gather_rows(int32_t heads, int32_t n_blocks, int32_t block, int32_t row_bytes,
                                            const void* src, const int64_t* src_stride_bytes, void* dst,
                                            const int64_t* dst_stride_bytes, const int32_t* row_order,
                                            void* cuda_stream) {
  return move_blocks(false, heads, n_blocks, block, row_bytes, src, src_stride_bytes, dst, dst_stride_bytes, row_order,
                     static_cast<cudaStream_t>(cuda_stream));
}

extern "C" waveal_status waveal_scatter_rows(int32_t heads, int32_t n_blocks, int32_t block, int32_t row_bytes,
                                             const void* src, const int64_t* src_stride_bytes, void* dst,
                                             const int64_t* dst_stride_bytes, const int32_t* row_order,
                                             void* cuda_stream) {
  return move_blocks(true, heads, n_blocks, block, row_bytes, src, src_stride_bytes, dst, dst_stride_bytes, row_order,
                     static_cast<cudaStream_t>(cuda_stream));
}
