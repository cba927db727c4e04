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
//                  all key blocks (pooled K streamed from L2, coalesced along j,
//                  packed fp32x2 FMAs over row pairs), then one warp per query
//                  block does an exact radix select of the topk-th largest key
//                  (keys in registers for nb <= 768) and an ordered ballot compaction.
#include "common.cuh"
#include "launch.h"

namespace sparkattn {

constexpr int kPoolThreads = 256;
constexpr int kTopkThreads = 320;  // 2 x 320 key-block slots per sweep (591 blocks of the 720P shape fit one sweep)
constexpr int kRowsPerCta = 8;     // query blocks per CTA; warps 0-7 select one row each

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

// Exact selection of the topk largest keys of one row by one warp (ties: lowest index first),
// written in ascending index order.  KeyAt(j) returns key j; the keys are visited several times.
// Only the key blocks jlo..jhi are candidates (the whole row without a causal window); the caller
// passes topk <= jhi - jlo + 1 and key_at returns 0 (below every real key) outside that range.
template <typename KeyAt>
__device__ __forceinline__ void select_row(KeyAt key_at, int nb, int jlo, int jhi, int topk, int lane,
                                           int32_t* __restrict__ dst) {
  // value of the topk-th largest key, one bit per pass from the top; bits above the highest bit in
  // which the row's keys differ are common to all keys and need no pass
  uint32_t kmin = 0xffffffffu, kmaxv = 0u;
  for (int j = jlo + lane; j <= jhi; j += 32) {
    const uint32_t kj = key_at(j);
    kmin = min(kmin, kj);
    kmaxv = max(kmaxv, kj);
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmaxv = __reduce_max_sync(0xffffffffu, kmaxv);
  const int top_bit = 31 - __clz(kmin ^ kmaxv);              // -1 when all keys are equal
  uint32_t thr = (top_bit >= 31) ? 0u : (kmaxv & ~((2u << max(top_bit, 0)) - 1u));
  if (top_bit < 0) thr = kmaxv;
  for (int bit = top_bit; bit >= 0; --bit) {
    const uint32_t cand = thr | (1u << bit);
    int cnt = 0;
    for (int j = lane; j < nb; j += 32) cnt += (key_at(j) >= cand);
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (cnt >= topk) thr = cand;
  }
  int ngreater = 0;
  for (int j = lane; j < nb; j += 32) ngreater += (key_at(j) > thr);
  ngreater = __reduce_add_sync(0xffffffffu, ngreater);
  const int ties_allowed = topk - ngreater;  // >= 1: lowest indices among the keys equal to thr

  int out = 0, ties_seen = 0;
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int base = 0; base < nb; base += 32) {
    const int j = base + lane;
    const bool valid = j >= jlo && j <= jhi;
    const uint32_t kj = valid ? key_at(j) : 0u;
    const bool tie = valid && (kj == thr);
    const uint32_t tie_ballot = __ballot_sync(0xffffffffu, tie);
    const int tie_rank = ties_seen + __popc(tie_ballot & lt_mask);
    const bool keep = valid && ((kj > thr) || (tie && tie_rank < ties_allowed));
    const uint32_t keep_ballot = __ballot_sync(0xffffffffu, keep);
    if (keep) dst[out + __popc(keep_ballot & lt_mask)] = j;
    out += __popc(keep_ballot);
    ties_seen += __popc(tie_ballot);
  }
}

constexpr int kKeysInRegs = 24;   // rows with nb <= 32 * 24 keep their keys in registers during the selection

template <int D, bool WINDOW>
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(const float* __restrict__ pq, const float* __restrict__ pkT, int32_t* __restrict__ kept_idx,
            int32_t* __restrict__ kept_cnt, int nb, int nbp, int topk, int groups_per_bh, int N, int blk_size,
            int frame_tokens, int window) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // pooled Q of the CTA's 8 query blocks, channel-major: s_pq[c][r], so that one 16-byte load
  // yields four rows of one channel as two packed fp32x2 operands
  float* s_pq = reinterpret_cast<float*>(smem_raw);                          // [D][kRowsPerCta]
  uint32_t* s_key = reinterpret_cast<uint32_t*>(s_pq + kRowsPerCta * D);     // [kRowsPerCta][nbp]

  const int64_t bh = blockIdx.x / groups_per_bh;
  const int i0 = (blockIdx.x % groups_per_bh) * kRowsPerCta;
  const int nrows = min(kRowsPerCta, nb - i0);

  for (int e = threadIdx.x; e < kRowsPerCta * D; e += kTopkThreads) {
    const int r = e / D, c = e % D;
    s_pq[c * kRowsPerCta + r] = (r < nrows) ? pq[(bh * nb + i0 + r) * D + c] : 0.0f;
  }
  __syncthreads();

  // scores: a thread owns kJT key blocks (j, j + kTopkThreads) and walks the channels in ascending
  // order for the CTA's 8 query blocks at once.  fma.rn.f32x2 is a pair of IEEE fmaf, so every
  // accumulator still sees exactly the chain a = fmaf(pq[i,c], pk[j,c], a), c ascending.
  const float* kcol = pkT + bh * D * (int64_t)nbp;
  const ulonglong2* s_pq2 = reinterpret_cast<const ulonglong2*>(s_pq);       // [D][kRowsPerCta / 4]
  constexpr int kJT = 2;
  constexpr int kPairs = kRowsPerCta / 2;
  for (int j0 = threadIdx.x; j0 < nb; j0 += kTopkThreads * kJT) {
    int jcl[kJT];
#pragma unroll
    for (int u = 0; u < kJT; ++u) jcl[u] = min(j0 + u * kTopkThreads, nb - 1);  // clamped: loads stay in range
    uint64_t acc[kJT][kPairs];
#pragma unroll
    for (int u = 0; u < kJT; ++u)
#pragma unroll
      for (int r = 0; r < kPairs; ++r) acc[u][r] = pack_f32x2(0.0f, 0.0f);
    constexpr int kCB = 16;  // channels per batch of loads (2 x 16 loads in flight per thread)
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += kCB) {
      float kv[kJT][kCB];
#pragma unroll
      for (int u = 0; u < kJT; ++u)
#pragma unroll
        for (int cc = 0; cc < kCB; ++cc) kv[u][cc] = __ldg(kcol + (int64_t)(c0 + cc) * nbp + jcl[u]);
#pragma unroll
      for (int cc = 0; cc < kCB; ++cc) {
        const ulonglong2 qa = s_pq2[(c0 + cc) * 2], qb = s_pq2[(c0 + cc) * 2 + 1];   // rows (0,1),(2,3) | (4,5),(6,7)
#pragma unroll
        for (int u = 0; u < kJT; ++u) {
          const uint64_t k2 = pack_f32x2(kv[u][cc], kv[u][cc]);
          acc[u][0] = ffma2(qa.x, k2, acc[u][0]);
          acc[u][1] = ffma2(qa.y, k2, acc[u][1]);
          acc[u][2] = ffma2(qb.x, k2, acc[u][2]);
          acc[u][3] = ffma2(qb.y, k2, acc[u][3]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kJT; ++u) {
      const int j = j0 + u * kTopkThreads;
      if (j < nb) {
#pragma unroll
        for (int r = 0; r < kPairs; ++r) {
          const float2 a = unpack_f32x2(acc[u][r]);
          s_key[(2 * r) * nbp + j] = score_key(a.x);
          s_key[(2 * r + 1) * nbp + j] = score_key(a.y);
        }
      }
    }
  }
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp >= nrows) return;   // (warps beyond the 8 rows of the CTA have no row)
  const uint32_t* key = s_key + warp * nbp;
  int32_t* dst = kept_idx + (bh * nb + i0 + warp) * (int64_t)topk;
  // Causal frame window (Sec. 1, auto-regressive extension): only the key blocks that hold a key some
  // row of this query block may attend to are candidates, a contiguous run jlo..jhi.
  int jlo = 0, jhi = nb - 1;
  if constexpr (WINDOW) {
    const int r0 = (i0 + warp) * blk_size, r1 = min((i0 + warp + 1) * blk_size, N) - 1;
    const int f0 = max(r0 / frame_tokens - window + 1, 0);
    const int kend = (int)min((long long)(r1 / frame_tokens + 1) * frame_tokens, (long long)N);
    jlo = (int)((long long)f0 * frame_tokens / blk_size);
    jhi = (kend - 1) / blk_size;
  }
  const int topk_all = topk;
  topk = min(topk, jhi - jlo + 1);
  auto in_range = [&](int j) { return WINDOW ? (j >= jlo && j <= jhi) : (j < nb); };
  if (nb <= 32 * kKeysInRegs) {
    uint32_t kr[kKeysInRegs];
#pragma unroll
    for (int u = 0; u < kKeysInRegs; ++u) {
      const int j = lane + 32 * u;
      kr[u] = in_range(j) ? key[j] : 0u;
    }
    // same algorithm as select_row, with the key loops unrolled over registers; a padding key
    // of 0 is below every candidate (candidates are >= 1) and is excluded by index where needed
    uint32_t kmin = 0xffffffffu, kmaxv = 0u;
#pragma unroll
    for (int u = 0; u < kKeysInRegs; ++u)
      if (in_range(lane + 32 * u)) { kmin = min(kmin, kr[u]); kmaxv = max(kmaxv, kr[u]); }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmaxv = __reduce_max_sync(0xffffffffu, kmaxv);
    const int top_bit = 31 - __clz(kmin ^ kmaxv);
    uint32_t thr = (top_bit >= 31) ? 0u : (kmaxv & ~((2u << max(top_bit, 0)) - 1u));
    if (top_bit < 0) thr = kmaxv;
    for (int bit = top_bit; bit >= 0; --bit) {
      const uint32_t cand = thr | (1u << bit);
      int cnt = 0;
#pragma unroll
      for (int u = 0; u < kKeysInRegs; ++u) cnt += (kr[u] >= cand);
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if (cnt >= topk) thr = cand;
    }
    int ngreater = 0;
#pragma unroll
    for (int u = 0; u < kKeysInRegs; ++u) ngreater += in_range(lane + 32 * u) && (kr[u] > thr);
    ngreater = __reduce_add_sync(0xffffffffu, ngreater);
    const int ties_allowed = topk - ngreater;
    int out = 0, ties_seen = 0;
    const uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
    for (int u = 0; u < kKeysInRegs; ++u) {
      if (32 * u < nb) {
        const int j = lane + 32 * u;
        const bool valid = in_range(j);
        const bool tie = valid && (kr[u] == thr);
        const uint32_t tie_ballot = __ballot_sync(0xffffffffu, tie);
        const int tie_rank = ties_seen + __popc(tie_ballot & lt_mask);
        const bool keep = valid && ((kr[u] > thr) || (tie && tie_rank < ties_allowed));
        const uint32_t keep_ballot = __ballot_sync(0xffffffffu, keep);
        if (keep) dst[out + __popc(keep_ballot & lt_mask)] = j;
        out += __popc(keep_ballot);
        ties_seen += __popc(tie_ballot);
      }
    }
  } else {
    select_row([&](int j) { return in_range(j) ? key[j] : 0u; }, nb, jlo, jhi, topk, lane, dst);
  }
  if constexpr (WINDOW)
    for (int t = topk + lane; t < topk_all; t += 32) dst[t] = -1;    // unused tail of a list cut short by the window
  if (lane == 0 && kept_cnt != nullptr) kept_cnt[bh * nb + i0 + warp] = topk;
}

int launch_select(const sparkattn_shape_t& s, const void* q, const void* k, int topk, int frame_tokens, int window,
                  int32_t* kept_idx, int32_t* kept_cnt, void* workspace, cudaStream_t stream) {
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
    auto kern = frame_tokens > 0 ? topk_kernel<128, true> : topk_kernel<128, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SPARKATTN_E_CUDA;
    kern<<<(unsigned)topk_ctas, kTopkThreads, smem, stream>>>(pq, pkT, kept_idx, kept_cnt, nb, nbp, topk, groups, s.N,
                                                             s.block, frame_tokens, window);
  } else if (s.d == 64) {
    pool_kernel<64><<<(unsigned)pool_ctas, kPoolThreads, 0, stream>>>(
        qb, kb, pq, pkT, s.H, s.N, s.block, nb, nbp, s.stride_b, s.stride_h, s.stride_n, n_items);
    auto kern = frame_tokens > 0 ? topk_kernel<64, true> : topk_kernel<64, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return SPARKATTN_E_CUDA;
    kern<<<(unsigned)topk_ctas, kTopkThreads, smem, stream>>>(pq, pkT, kept_idx, kept_cnt, nb, nbp, topk, groups, s.N,
                                                             s.block, frame_tokens, window);
  } else {
    return SPARKATTN_E_UNSUPPORTED_SHAPE;
  }
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

}  // namespace sparkattn
