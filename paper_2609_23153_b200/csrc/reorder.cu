// sparkattn_brick_layout / sparkattn_gather_tokens: tokens stored brick by brick.
//
// The paper partitions the token sequence into contiguous blocks (Sec. 2) and leaves the order of
// the tokens open; in raster order a 128-token block of a 45 x 80 frame is a strip of 1.6 grid rows.
// Here the (T, Hg, Wg) grid is cut into bricks of bt x bh x bw cells (bricks at the far faces are cut
// to what the grid holds), bricks follow one another in raster order of the brick grid, the cells of
// a brick in raster order inside it, and every brick takes one whole block: its cells first, padding
// rows after them.  A block is then a compact box of the video, at the price of padding wherever
// bt * bh * bw < block or a brick is cut short.  The other calls take the per-block count of real
// tokens (block_valid) so that padding rows are neither keys nor part of a pooled mean.
//
//   brick_layout_kernel  one thread per raster token: closed-form padded position (the bricks before
//                        it are counted by brick index, so no prefix sums are needed); writes the
//                        gather index (raster token at each padded position; padding keeps the -1 a
//                        memset put there), the scatter index and the per-brick token count.
//   gather_tokens_kernel out[b,h,i,:] = x[b,h,index[i],:] (zero row for index -1); a CTA moves 128
//                        (d = 128) or 256 (d = 64) consecutive rows of one (batch, head) as 16-byte
//                        pieces, 8 in flight per thread; bound by HBM (2 bytes read + 2 written per
//                        element).
#include "common.cuh"
#include "launch.h"

namespace sparkattn {

__global__ void __launch_bounds__(256)
brick_layout_kernel(int T, int Hg, int Wg, int bt, int bh, int bw, int block, int32_t* __restrict__ gather,
                    int32_t* __restrict__ block_valid, int32_t* __restrict__ scatter) {
  const int64_t N = (int64_t)T * Hg * Wg;
  const int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= N) return;
  const int x = (int)(n % Wg), y = (int)((n / Wg) % Hg), t = (int)(n / ((int64_t)Wg * Hg));
  const int i = t / bt, j = y / bh, k = x / bw;
  const int nbh = (Hg + bh - 1) / bh, nbw = (Wg + bw - 1) / bw;
  const int et = min(bt, T - i * bt), eh = min(bh, Hg - j * bh), ew = min(bw, Wg - k * bw);   // extents of this brick
  const int64_t brick = ((int64_t)i * nbh + j) * nbw + k;
  const int within = ((t - i * bt) * eh + (y - j * bh)) * ew + (x - k * bw);
  const int64_t p = brick * block + within;
  if (gather) gather[p] = (int32_t)n;
  if (scatter) scatter[n] = (int32_t)p;
  if (block_valid && within == 0) block_valid[brick] = et * eh * ew;
}

constexpr int kGatherThreads = 256, kGatherUnroll = 8;

// One CTA moves kGatherUnroll * 256 / PIECES consecutive token rows of one (batch, head): a thread keeps its
// 16-byte column of the row and steps over the rows, all loads issued before the first store.
template <int PIECES>   // 16-byte pieces per token row: 16 (d = 128) or 8 (d = 64)
__global__ void __launch_bounds__(kGatherThreads)
gather_tokens_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ index, uint4* __restrict__ out, int H,
                     int n_src, int n_dst, int64_t src_b, int64_t src_h, int64_t src_n, int64_t dst_b, int64_t dst_h,
                     int64_t dst_n /* strides in 16-byte pieces */, int chunks_per_bh, int32_t* __restrict__ status) {
  constexpr int kRowsPerPass = kGatherThreads / PIECES;
  constexpr int kRowsPerCta = kRowsPerPass * kGatherUnroll;
  const int bh = blockIdx.x / chunks_per_bh;
  const int row0 = (blockIdx.x - bh * chunks_per_bh) * kRowsPerCta + threadIdx.x / PIECES;
  const int piece = threadIdx.x % PIECES;
  const int b = bh / H, h = bh - b * H;
  const uint4* xs = x + b * src_b + h * src_h + piece;
  uint4* os = out + b * dst_b + h * dst_h + piece;
  uint4 v[kGatherUnroll];
#pragma unroll
  for (int u = 0; u < kGatherUnroll; ++u) {
    const int i = row0 + u * kRowsPerPass;
    v[u] = make_uint4(0u, 0u, 0u, 0u);
    if (i < n_dst) {
      const int src = __ldg(index + i);
      if ((unsigned)src < (unsigned)n_src) v[u] = __ldg(xs + (int64_t)src * src_n);
      else if (src != -1) report_status(status, SPARKATTN_E_BAD_INDEX, src);     // the row is written as zeros
    }
  }
#pragma unroll
  for (int u = 0; u < kGatherUnroll; ++u) {
    const int i = row0 + u * kRowsPerPass;
    if (i < n_dst) os[(int64_t)i * dst_n] = v[u];
  }
}

int launch_brick_layout(const int32_t* grid, const int32_t* brick, int block, int32_t* gather, int32_t* block_valid,
                        int32_t* scatter, cudaStream_t stream) {
  const int64_t N = (int64_t)grid[0] * grid[1] * grid[2];
  const int64_t bricks = (int64_t)((grid[0] + brick[0] - 1) / brick[0]) * ((grid[1] + brick[1] - 1) / brick[1]) *
                         ((grid[2] + brick[2] - 1) / brick[2]);
  if (gather && cudaMemsetAsync(gather, 0xff, (size_t)bricks * block * sizeof(int32_t), stream) != cudaSuccess)
    return SPARKATTN_E_CUDA;                                              // every position padding (-1) until written
  const unsigned ctas = (unsigned)((N + 255) / 256);
  brick_layout_kernel<<<ctas, 256, 0, stream>>>(grid[0], grid[1], grid[2], brick[0], brick[1], brick[2], block, gather,
                                                block_valid, scatter);
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

int launch_gather_tokens(const sparkattn_shape_t& src, const void* x, const sparkattn_shape_t& dst, const int32_t* index,
                         void* out, void* workspace, cudaStream_t stream) {
  const int pieces = dst.d * 2 / 16;
  const int rows_per_cta = kGatherThreads / pieces * kGatherUnroll;
  const int chunks = (dst.N + rows_per_cta - 1) / rows_per_cta;
  const int64_t ctas = (int64_t)dst.B * dst.H * chunks;
  if (ctas > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  int32_t* status = static_cast<int32_t*>(workspace);
  const uint4* xs = static_cast<const uint4*>(x);
  uint4* os = static_cast<uint4*>(out);
  if (dst.d == 128)
    gather_tokens_kernel<16><<<(unsigned)ctas, kGatherThreads, 0, stream>>>(
        xs, index, os, dst.H, src.N, dst.N, src.stride_b / 8, src.stride_h / 8, src.stride_n / 8, dst.stride_b / 8,
        dst.stride_h / 8, dst.stride_n / 8, chunks, status);
  else
    gather_tokens_kernel<8><<<(unsigned)ctas, kGatherThreads, 0, stream>>>(
        xs, index, os, dst.H, src.N, dst.N, src.stride_b / 8, src.stride_h / 8, src.stride_n / 8, dst.stride_b / 8,
        dst.stride_h / 8, dst.stride_n / 8, chunks, status);
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

}  // namespace sparkattn
