// sparkattn_select: pooled block scores + top-k kept-block lists.
//
// The paper's selector M_phi (Sec. 2, Sec. 4.1) is left open ("top-k
// selection, blockwise scores"); the rule implemented here is
//   pooled mean of every token block (fp32, tokens added in ascending order,
//   one IEEE divide), score(i,j) = fmaf chain over channels, keep the topk
//   key blocks first under (score descending, index ascending), emit ascending.
// Every floating-point step has a fixed order so that the result is defined
// bit for bit; this is why scoring runs on the FMA pipe and not on tensor cores.
//
// Two kernels:
//   pool_kernel    one warp per (tensor, batch, head, block); reads Q and K once
//                  from HBM (the only HBM-heavy step: 2 bytes per element) and
//                  writes pooled Q [BH][nb][d] and pooled K transposed [BH][d][nbp].
//   topk_kernel    one CTA per 8 query blocks of one (batch, head): scores against
//                  all key blocks (pooled K streamed from L2, coalesced along j),
//                  then one warp per query block does an exact radix select of the
//                  topk-th largest key and an ordered ballot compaction.
#include "common.cuh"
#include "launch.h"

namespace sparkattn {

constexpr int kPoolThreads = 256;
constexpr int kTopkThreads = 256;
constexpr int kRowsPerCta = kTopkThreads / 32;  // query blocks per CTA, one warp each

static inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

size_t select_workspace_bytes(const sparkattn_shape_t& s) {
  const int nb = (s.N + s.block - 1) / s.block;
  const int nbp = round_up(nb, 32);
  const size_t bh = (size_t)s.B * s.H;
  return kWorkspaceHeaderBytes + bh * nb * s.d * sizeof(float) + bh * s.d * nbp * sizeof(float);
}

template <int D>
__global__ void __launch_bounds__(kPoolThreads)
pool_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, float* __restrict__ pq,
            float* __restrict__ pkT, int H, int N, int blk_size, int nb, int nbp, int64_t stride_b,
            int64_t stride_h, int64_t stride_n, int64_t n_items /* B*H*nb */) {
  constexpr int VEC = D / 32;  // channels per lane: 4 (8-byte loads) or 2 (4-byte loads)
  const int lane = threadIdx.x & 31;
  const int64_t gw = (int64_t)blockIdx.x * (kPoolThreads / 32) + (threadIdx.x >> 5);
  if (gw >= 2 * n_items) return;
  const bool is_k = gw >= n_items;
  const int64_t item = is_k ? gw - n_items : gw;
  const int blk = (int)(item % nb);
  const int64_t bh = item / nb;
  const int h = (int)(bh % H), b = (int)(bh / H);
  const int row0 = blk * blk_size;
  const int nvalid = min(blk_size, N - row0);
  const __nv_bfloat16* src = (is_k ? k : q) + b * stride_b + h * stride_h + (int64_t)row0 * stride_n + lane * VEC;

  float sum[VEC];
#pragma unroll
  for (int c = 0; c < VEC; ++c) sum[c] = 0.0f;

  constexpr int U = 16;  // rows in flight per lane
  int t = 0;
  for (; t + U <= nvalid; t += U) {
    float x[U][VEC];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const __nv_bfloat16* p = src + (int64_t)(t + u) * stride_n;
      if constexpr (VEC == 4) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(p));
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
        const float2 c = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
        x[u][0] = a.x; x[u][1] = a.y; x[u][2] = c.x; x[u][3] = c.y;
      } else {
        const uint32_t raw = __ldg(reinterpret_cast<const uint32_t*>(p));
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw));
        x[u][0] = a.x; x[u][1] = a.y;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int c = 0; c < VEC; ++c) sum[c] = __fadd_rn(sum[c], x[u][c]);
  }
  for (; t < nvalid; ++t) {
    const __nv_bfloat16* p = src + (int64_t)t * stride_n;
#pragma unroll
    for (int c = 0; c < VEC; ++c) sum[c] = __fadd_rn(sum[c], __bfloat162float(p[c]));
  }
  const float nv = (float)nvalid;
#pragma unroll
  for (int c = 0; c < VEC; ++c) {
    const float mean = __fdiv_rn(sum[c], nv);
    const int ch = lane * VEC + c;
    if (is_k) pkT[(bh * D + ch) * nbp + blk] = mean;
    else pq[(bh * nb + blk) * D + ch] = mean;
  }
}

// Order-preserving map fp32 -> uint32 (larger float = larger key); -0 is folded onto +0.
__device__ __forceinline__ uint32_t score_key(float s) {
  const uint32_t u = __float_as_uint(s + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <int D>
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ pq, const float* __restrict__ pkT, int32_t* __restrict__ kept_idx,
            int32_t* __restrict__ kept_cnt, int nb, int nbp, int topk, int groups_per_bh) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_pq = reinterpret_cast<float*>(smem_raw);                          // [kRowsPerCta][D], 16-byte aligned
  uint32_t* s_key = reinterpret_cast<uint32_t*>(s_pq + kRowsPerCta * D);     // [kRowsPerCta][nbp]

  const int64_t bh = blockIdx.x / groups_per_bh;
  const int i0 = (blockIdx.x % groups_per_bh) * kRowsPerCta;
  const int nrows = min(kRowsPerCta, nb - i0);

  for (int e = threadIdx.x; e < kRowsPerCta * D; e += kTopkThreads) {
    const int r = e / D;
    s_pq[e] = (r < nrows) ? pq[(bh * nb + i0 + r) * D + (e % D)] : 0.0f;
  }
  __syncthreads();

  // scores: a thread owns up to kJT key blocks (j, j + 256, j + 512) and walks the channels in
  // ascending order for the CTA's 8 query blocks at once; pooled Q comes from shared memory as
  // broadcast 16-byte loads, pooled K from L2 coalesced along j.
  const float* kcol = pkT + bh * D * (int64_t)nbp;
  const float4* s_pq4 = reinterpret_cast<const float4*>(s_pq);
  constexpr int kJT = 3;
  for (int j0 = threadIdx.x; j0 < nb; j0 += kTopkThreads * kJT) {
    int jcl[kJT];
#pragma unroll
    for (int u = 0; u < kJT; ++u) jcl[u] = min(j0 + u * kTopkThreads, nb - 1);  // clamped: loads stay in range
    float acc[kJT][kRowsPerCta];
#pragma unroll
    for (int u = 0; u < kJT; ++u)
#pragma unroll
      for (int r = 0; r < kRowsPerCta; ++r) acc[u][r] = 0.0f;
#pragma unroll 2
    for (int c4 = 0; c4 < D / 4; ++c4) {
      float4 qv[kRowsPerCta];
#pragma unroll
      for (int r = 0; r < kRowsPerCta; ++r) qv[r] = s_pq4[r * (D / 4) + c4];
#pragma unroll
      for (int u = 0; u < kJT; ++u) {
        const float* kp = kcol + (int64_t)(4 * c4) * nbp + jcl[u];
        const float k0 = __ldg(kp), k1 = __ldg(kp + nbp), k2 = __ldg(kp + 2 * nbp), k3 = __ldg(kp + 3 * nbp);
#pragma unroll
        for (int r = 0; r < kRowsPerCta; ++r) {
          float a = acc[u][r];
          a = __fmaf_rn(qv[r].x, k0, a);
          a = __fmaf_rn(qv[r].y, k1, a);
          a = __fmaf_rn(qv[r].z, k2, a);
          a = __fmaf_rn(qv[r].w, k3, a);
          acc[u][r] = a;
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kJT; ++u) {
      const int j = j0 + u * kTopkThreads;
      if (j < nb) {
#pragma unroll
        for (int r = 0; r < kRowsPerCta; ++r) s_key[r * nbp + j] = score_key(acc[u][r]);
      }
    }
  }
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp >= nrows) return;
  const uint32_t* key = s_key + warp * nbp;

  // exact value of the topk-th largest key, one bit per pass from the top; bits above the
  // highest bit in which the row's keys differ are common to all keys and need no pass
  uint32_t kmin = 0xffffffffu, kmaxv = 0u;
  for (int j = lane; j < nb; j += 32) {
    kmin = min(kmin, key[j]);
    kmaxv = max(kmaxv, key[j]);
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmaxv = __reduce_max_sync(0xffffffffu, kmaxv);
  const uint32_t diff = kmin ^ kmaxv;
  const int top_bit = 31 - __clz(diff);                       // -1 when all keys are equal
  uint32_t thr = (top_bit >= 31) ? 0u : (kmaxv & ~((2u << max(top_bit, 0)) - 1u));
  if (top_bit < 0) thr = kmaxv;
  for (int bit = top_bit; bit >= 0; --bit) {
    const uint32_t cand = thr | (1u << bit);
    int cnt = 0;
    for (int j = lane; j < nb; j += 32) cnt += (key[j] >= cand);
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (cnt >= topk) thr = cand;
  }
  int ngreater = 0;
  for (int j = lane; j < nb; j += 32) ngreater += (key[j] > thr);
  ngreater = __reduce_add_sync(0xffffffffu, ngreater);
  const int ties_allowed = topk - ngreater;  // >= 1: lowest indices among the keys equal to thr

  int32_t* dst = kept_idx + (bh * nb + i0 + warp) * (int64_t)topk;
  int out = 0, ties_seen = 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int base = 0; base < nb; base += 32) {
    const int j = base + lane;
    const uint32_t kj = (j < nb) ? key[j] : 0u;
    const bool valid = j < nb;
    const bool tie = valid && (kj == thr);
    const uint32_t tie_ballot = __ballot_sync(0xffffffffu, tie);
    const int tie_rank = ties_seen + __popc(tie_ballot & lt_mask);
    const bool keep = valid && ((kj > thr) || (tie && tie_rank < ties_allowed));
    const uint32_t keep_ballot = __ballot_sync(0xffffffffu, keep);
    if (keep) dst[out + __popc(keep_ballot & lt_mask)] = j;
    out += __popc(keep_ballot);
    ties_seen += __popc(tie_ballot);
  }
  if (lane == 0 && kept_cnt != nullptr) kept_cnt[bh * nb + i0 + warp] = topk;
}

int launch_select(const sparkattn_shape_t& s, const void* q, const void* k, int topk, int32_t* kept_idx,
                  int32_t* kept_cnt, void* workspace, cudaStream_t stream) {
  const int nb = (s.N + s.block - 1) / s.block;
  const int nbp = round_up(nb, 32);
  if (nb > kSelectMaxBlocks) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const int64_t bh = (int64_t)s.B * s.H;
  const int64_t n_items = bh * nb;
  float* pq = reinterpret_cast<float*>(static_cast<char*>(workspace) + kWorkspaceHeaderBytes);
  float* pkT = pq + n_items * s.d;
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);

  const int64_t pool_ctas = (2 * n_items + kPoolThreads / 32 - 1) / (kPoolThreads / 32);
  const int groups = (nb + kRowsPerCta - 1) / kRowsPerCta;
  const int64_t topk_ctas = bh * groups;
  if (pool_ctas > 0x7fffffffLL || topk_ctas > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const size_t smem = (size_t)kRowsPerCta * s.d * sizeof(float) + (size_t)kRowsPerCta * nbp * sizeof(uint32_t);

  if (s.d == 128) {
    pool_kernel<128><<<(unsigned)pool_ctas, kPoolThreads, 0, stream>>>(
        qb, kb, pq, pkT, s.H, s.N, s.block, nb, nbp, s.stride_b, s.stride_h, s.stride_n, n_items);
    if (cudaFuncSetAttribute(topk_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return SPARKATTN_E_CUDA;
    topk_kernel<128><<<(unsigned)topk_ctas, kTopkThreads, smem, stream>>>(pq, pkT, kept_idx, kept_cnt, nb, nbp,
                                                                          topk, groups);
  } else if (s.d == 64) {
    pool_kernel<64><<<(unsigned)pool_ctas, kPoolThreads, 0, stream>>>(
        qb, kb, pq, pkT, s.H, s.N, s.block, nb, nbp, s.stride_b, s.stride_h, s.stride_n, n_items);
    if (cudaFuncSetAttribute(topk_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
      return SPARKATTN_E_CUDA;
    topk_kernel<64><<<(unsigned)topk_ctas, kTopkThreads, smem, stream>>>(pq, pkT, kept_idx, kept_cnt, nb, nbp,
                                                                         topk, groups);
  } else {
    return SPARKATTN_E_UNSUPPORTED_SHAPE;
  }
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

}  // namespace sparkattn
