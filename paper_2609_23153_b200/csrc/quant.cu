// sparkattn_quant_fp8: per-(batch, head, token block) absmax scale + E4M3
// encode in one pass over memory (paper Sec. 4.3: FP8 E4M3, scaling and
// casting fused in a single kernel).
//
// One CTA owns one token block: it loads the block's bf16 elements into
// registers once (16-byte loads, rows contiguous), reduces |x| to the block
// maximum, then scales, encodes (cvt.rn.satfinite.e4m3x2.f32) and stores from
// the same registers, so HBM sees one read of x and one write of the codes:
// 3 bytes per element.
#include <cuda_fp8.h>

#include "common.cuh"
#include "launch.h"

namespace sparkattn {

constexpr int kQuantThreads = 256;

// POOL: the same pass also produces the block's pooled mean for the selection (Sec. 4.3 fuses scaling and
// casting into one pass over memory; with the pooling in it as well, Q and K are read from HBM once for
// selection and quantisation together).  The selection's pooled sum is a chain of fp32 additions over the
// block's tokens in ascending order, one chain per channel, so it cannot be spread over the threads that hold
// the rows: the block is parked in shared memory on the way and thread c walks channel c through it while the
// other warps encode.  pooled: fp32 [B*H][nb][D] (query side) or transposed [B*H][D][nbp] (key side).
template <int D, int BLK, bool POOL>
__global__ void __launch_bounds__(kQuantThreads, 3)
quant_fp8_kernel(const __nv_bfloat16* __restrict__ x, uint8_t* __restrict__ codes, float* __restrict__ scales,
                 int H, int N, int nb, int64_t stride_b, int64_t stride_h, int64_t stride_n,
                 float* __restrict__ pooled, int pooled_transposed, int nbp) {
  constexpr int kChunksPerRow = D / 8;                      // 16-byte chunks per token row
  constexpr int kChunks = BLK * kChunksPerRow;              // chunks per token block
  constexpr int kPerThread = kChunks / kQuantThreads;       // 8 for (128,128), 2 for (64,64)
  static_assert(kChunks % kQuantThreads == 0, "block must split evenly over the CTA");

  const int blk = blockIdx.x % nb;
  const int bh = blockIdx.x / nb;
  const int h = bh % H, b = bh / H;
  const int row0 = blk * BLK;
  const int nvalid = min(BLK, N - row0);
  const int64_t base = b * stride_b + h * stride_h;

  uint4 v[kPerThread];
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int ci = threadIdx.x + i * kQuantThreads;
    const int r = ci / kChunksPerRow, cc = ci % kChunksPerRow;
    if (r < nvalid) {
      v[i] = __ldg(reinterpret_cast<const uint4*>(x + base + (int64_t)(row0 + r) * stride_n + cc * 8));
    } else {
      v[i] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  __shared__ __align__(16) __nv_bfloat16 s_tile[POOL ? BLK * D : 8];
  if constexpr (POOL) {
#pragma unroll
    for (int i = 0; i < kPerThread; ++i)
      reinterpret_cast<uint4*>(s_tile)[threadIdx.x + i * kQuantThreads] = v[i];     // [row][channel], conflict-free
  }
#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v[i]);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(p[j]);
      amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
    }
  }
  __shared__ float s_red[kQuantThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = s_red[0];
#pragma unroll
  for (int w = 1; w < kQuantThreads / 32; ++w) amax = fmaxf(amax, s_red[w]);
  amax = fmaxf(amax, 1e-12f);
  const float inv = __fdiv_rn(448.0f, amax);
  if (threadIdx.x == 0) scales[(int64_t)bh * nb + blk] = __fdiv_rn(amax, 448.0f);

#pragma unroll
  for (int i = 0; i < kPerThread; ++i) {
    const int ci = threadIdx.x + i * kQuantThreads;
    const int r = ci / kChunksPerRow, cc = ci % kChunksPerRow;
    if (r >= nvalid) continue;
    const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v[i]);
    uint32_t w[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const float2 f0 = __bfloat1622float2(p[2 * j]);
      const float2 f1 = __bfloat1622float2(p[2 * j + 1]);
      const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(f0.x, inv), __fmul_rn(f0.y, inv)),
                                                    __NV_SATFINITE, __NV_E4M3);
      const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(f1.x, inv), __fmul_rn(f1.y, inv)),
                                                    __NV_SATFINITE, __NV_E4M3);
      w[j] = lo | (hi << 16);
    }
    *reinterpret_cast<uint2*>(codes + base + (int64_t)(row0 + r) * stride_n + cc * 8) = make_uint2(w[0], w[1]);
  }
  if constexpr (POOL) {
    // (the __syncthreads of the absmax reduction made the tile visible)
    if (threadIdx.x < D) {
      const int c = threadIdx.x;
      float sum = 0.0f;
      constexpr int U = 8;     // rows fetched ahead of the addition chain
      int r = 0;
      for (; r + U <= nvalid; r += U) {
        float xr[U];
#pragma unroll
        for (int u = 0; u < U; ++u) xr[u] = __bfloat162float(s_tile[(r + u) * D + c]);
#pragma unroll
        for (int u = 0; u < U; ++u) sum = __fadd_rn(sum, xr[u]);
      }
      for (; r < nvalid; ++r) sum = __fadd_rn(sum, __bfloat162float(s_tile[r * D + c]));
      const float mean = __fdiv_rn(sum, (float)nvalid);
      if (pooled_transposed) pooled[((int64_t)bh * D + c) * nbp + blk] = mean;
      else pooled[((int64_t)bh * nb + blk) * D + c] = mean;
    }
  }
}

// Per-token variant: a token row (d channels) is spread over 4 lanes; lane c of the group takes the
// 16-byte chunks c, c + 4, ... of the row, so that one load instruction of the warp covers 64
// contiguous bytes of each of 8 rows.  A warp walks kTokenSteps steps of 8 rows with all loads issued
// first (128 bytes in flight per thread).  absmax over the lane's chunks, two shuffles inside the lane
// group, then the two IEEE divisions once per row (they are a third of the instructions when a lane
// holds a single chunk), encode and store from the same registers: one HBM read, one write.
constexpr int kTokenSteps = 2;
constexpr int kTokenLanes = 4;                   // lanes per row
constexpr int kTokenRows = 32 / kTokenLanes;     // rows per warp step

template <int D>
__global__ void __launch_bounds__(kQuantThreads, 3)
quant_fp8_token_kernel(const __nv_bfloat16* __restrict__ x, uint8_t* __restrict__ codes, float* __restrict__ scales,
                       int H, int N, int64_t stride_b, int64_t stride_h, int64_t stride_n, int64_t n_rows) {
  constexpr int CPL = D / 8 / kTokenLanes;       // chunks per lane: 4 (d=128) or 2 (d=64)
  const int lane = threadIdx.x & 31;
  const int sub = lane / kTokenLanes, chunk = lane % kTokenLanes;
  const int64_t warp_id = (int64_t)blockIdx.x * (kQuantThreads / 32) + (threadIdx.x >> 5);
  const int64_t row0 = warp_id * (kTokenSteps * kTokenRows);
  uint4 v[kTokenSteps][CPL];
  int64_t off[kTokenSteps];
  // (batch, head, token) of this lane's first row: divisions once, then the rows just count up
  const uint32_t first = (uint32_t)(row0 + sub);            // n_rows < 2^31 (checked by the launcher)
  const uint32_t bh0 = first / (uint32_t)N;
  int n = (int)(first - bh0 * (uint32_t)N);
  int b = (int)(bh0 / (uint32_t)H), h = (int)(bh0 - (uint32_t)b * (uint32_t)H);
#pragma unroll
  for (int u = 0; u < kTokenSteps; ++u) {
    const int64_t r = row0 + u * kTokenRows + sub;
    off[u] = b * stride_b + h * stride_h + (int64_t)n * stride_n + chunk * 8;
    n += kTokenRows;
    while (n >= N) {
      n -= N;
      if (++h == H) { h = 0; ++b; }
    }
#pragma unroll
    for (int c = 0; c < CPL; ++c)
      v[u][c] = (r < n_rows) ? __ldg(reinterpret_cast<const uint4*>(x + off[u] + c * (kTokenLanes * 8)))
                             : make_uint4(0u, 0u, 0u, 0u);
  }
#pragma unroll
  for (int u = 0; u < kTokenSteps; ++u) {
    const int64_t r = row0 + u * kTokenRows + sub;
    float f[CPL][8];
    float amax = 0.0f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
      const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&v[u][c]);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 t = __bfloat1622float2(p2[j]);
        f[c][2 * j] = t.x;
        f[c][2 * j + 1] = t.y;
        amax = fmaxf(amax, fmaxf(fabsf(t.x), fabsf(t.y)));
      }
    }
#pragma unroll
    for (int o = kTokenLanes / 2; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    amax = fmaxf(amax, 1e-12f);
    const float inv = __fdiv_rn(448.0f, amax);
    if (r >= n_rows) continue;
    if (chunk == 0) scales[r] = __fdiv_rn(amax, 448.0f);
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
      uint32_t w[2];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(f[c][4 * j], inv), __fmul_rn(f[c][4 * j + 1], inv)),
                                                      __NV_SATFINITE, __NV_E4M3);
        const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(__fmul_rn(f[c][4 * j + 2], inv), __fmul_rn(f[c][4 * j + 3], inv)),
                                                      __NV_SATFINITE, __NV_E4M3);
        w[j] = lo | (hi << 16);
      }
      *reinterpret_cast<uint2*>(codes + off[u] + c * (kTokenLanes * 8)) = make_uint2(w[0], w[1]);
    }
  }
}

int launch_quant_fp8_per_token(const sparkattn_shape_t& s, const void* x, uint8_t* codes, float* scales,
                               cudaStream_t stream) {
  const int64_t n_rows = (int64_t)s.B * s.H * s.N;
  if (n_rows >= (1LL << 31) - 4096) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const int64_t rows_per_cta = (kQuantThreads / 32) * kTokenSteps * kTokenRows;
  const int64_t ctas = (n_rows + rows_per_cta - 1) / rows_per_cta;
  if (ctas > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
  if (s.d == 128) {
    quant_fp8_token_kernel<128><<<(unsigned)ctas, kQuantThreads, 0, stream>>>(
        xb, codes, scales, s.H, s.N, s.stride_b, s.stride_h, s.stride_n, n_rows);
  } else if (s.d == 64) {
    quant_fp8_token_kernel<64><<<(unsigned)ctas, kQuantThreads, 0, stream>>>(
        xb, codes, scales, s.H, s.N, s.stride_b, s.stride_h, s.stride_n, n_rows);
  } else {
    return SPARKATTN_E_UNSUPPORTED_SHAPE;
  }
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

template <bool POOL>
static int launch_quant_fp8_t(const sparkattn_shape_t& s, const void* x, uint8_t* codes, float* scales, float* pooled,
                              int pooled_transposed, cudaStream_t stream) {
  const int nb = (s.N + s.block - 1) / s.block;
  const int nbp = (nb + 31) / 32 * 32;
  const long long ctas = (long long)s.B * s.H * nb;
  if (ctas > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
  if (s.d == 128 && s.block == 128) {
    quant_fp8_kernel<128, 128, POOL><<<(unsigned)ctas, kQuantThreads, 0, stream>>>(
        xb, codes, scales, s.H, s.N, nb, s.stride_b, s.stride_h, s.stride_n, pooled, pooled_transposed, nbp);
  } else if (s.d == 128 && s.block == 64) {
    quant_fp8_kernel<128, 64, POOL><<<(unsigned)ctas, kQuantThreads, 0, stream>>>(
        xb, codes, scales, s.H, s.N, nb, s.stride_b, s.stride_h, s.stride_n, pooled, pooled_transposed, nbp);
  } else if (s.d == 64 && s.block == 64) {
    quant_fp8_kernel<64, 64, POOL><<<(unsigned)ctas, kQuantThreads, 0, stream>>>(
        xb, codes, scales, s.H, s.N, nb, s.stride_b, s.stride_h, s.stride_n, pooled, pooled_transposed, nbp);
  } else {
    return SPARKATTN_E_UNSUPPORTED_SHAPE;
  }
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

int launch_quant_fp8(const sparkattn_shape_t& s, const void* x, uint8_t* codes, float* scales,
                     cudaStream_t stream) {
  return launch_quant_fp8_t<false>(s, x, codes, scales, nullptr, 0, stream);
}

// pooled: the selection workspace's pooled-Q or pooled-K region (select.cu lays it out)
int launch_quant_fp8_pooled(const sparkattn_shape_t& s, const void* x, uint8_t* codes, float* scales, float* pooled,
                            bool key_side, cudaStream_t stream) {
  return launch_quant_fp8_t<true>(s, x, codes, scales, pooled, key_side ? 1 : 0, stream);
}

}  // namespace sparkattn
