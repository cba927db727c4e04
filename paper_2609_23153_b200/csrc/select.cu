// sparkattn_select: pooled block scores + top-k kept-block lists.
//
// The paper's selector M_phi (Sec. 2, Sec. 4.1) is left open (it lists kinds of
// selectors, top-k over per-block scores among them); the rule implemented here is
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
//   topk_kernel    one CTA per 16 (8 for very long sequences) query blocks of one
//                  (batch, head): scores against all key blocks as a 16 x 4 register
//                  tile per thread (pooled K streamed from L2 in 16-byte loads along j,
//                  packed fp32x2 FMAs over row pairs), then one warp per query block
//                  does an exact radix select of the topk-th largest key (keys in
//                  registers for nb <= 1280) and an ordered ballot compaction.
#include "common.cuh"
#include "launch.h"

namespace sparkattn {

constexpr int kPoolThreads = 256;
constexpr int kTopkThreads = 160;  // 4 x 160 key-block slots per sweep (591 blocks of the 720P shape fit one sweep)

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
            int64_t stride_h, int64_t stride_n, int64_t n_items /* B*H*nb */,
            const int32_t* __restrict__ block_valid /* [nb] real tokens per block, or NULL */) {
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
  int nvalid = min(blk_size, N - row0);
  if (block_valid != nullptr) nvalid = max(1, min(nvalid, __ldg(block_valid + blk)));   // bricks padded to whole blocks
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

// select_row with the row's keys held in KR registers per lane (nb <= 32 * KR): the key loops unroll
// over registers.  Keys outside the candidate range are held as 0, below every candidate (candidates
// are >= 1).
//
// The threshold (the topk-th largest key) is first sought among the four largest keys of every lane,
// 128 values: their topk-th largest, T, never exceeds the true threshold, and when no lane holds more
// than four keys >= T every key >= T is among the 128, so T is the true threshold.  The bitwise search
// then costs 4 compares per pass instead of KR.  Otherwise (a lane with five such keys, or topk > 128)
// the search runs over all KR keys.  Either way the threshold is exact; only the cost differs.
template <int KR, bool WINDOW>
__device__ __forceinline__ void select_row_regs(const uint32_t* __restrict__ key, int nb, int jlo, int jhi, int topk,
                                                int lane, int32_t* __restrict__ dst) {
  constexpr uint32_t kFull = 0xffffffffu;
  auto in_range = [&](int j) { return WINDOW ? (j >= jlo && j <= jhi) : (j < nb); };
  uint32_t kr[KR];
#pragma unroll
  for (int u = 0; u < KR; ++u) {
    const int j = lane + 32 * u;
    kr[u] = in_range(j) ? key[j] : 0u;
  }
  // sorted four largest keys of the lane
  uint32_t m1 = 0u, m2 = 0u, m3 = 0u, m4 = 0u;
#pragma unroll
  for (int u = 0; u < KR; ++u) {
    uint32_t x = kr[u], t;
    t = min(m1, x); m1 = max(m1, x); x = t;
    t = min(m2, x); m2 = max(m2, x); x = t;
    t = min(m3, x); m3 = max(m3, x); x = t;
    m4 = max(m4, x);
  }
  const uint32_t kmaxv = __reduce_max_sync(kFull, m1);
  uint32_t thr = 0u;
  bool exact = false;
  int nge = 0;
  if (topk <= 128) {
    // T lies between the smallest lane maximum (32 >= topk values are at least that) and the row maximum;
    // the bits above the highest bit in which the two differ are common to both and need no pass
    const uint32_t lo = (topk <= 32) ? __reduce_min_sync(kFull, m1) : 0u;
    const int top_bit = 31 - __clz(lo ^ kmaxv);              // -1 when the two are equal
    thr = (top_bit >= 31) ? 0u : (kmaxv & ~((2u << max(top_bit, 0)) - 1u));
    if (top_bit < 0) thr = kmaxv;
    for (int bit = top_bit; bit >= 0; --bit) {
      const uint32_t cand = thr | (1u << bit);
      int cnt = (m1 >= cand) + (m2 >= cand) + (m3 >= cand) + (m4 >= cand);
      cnt = __reduce_add_sync(kFull, cnt);
      if (cnt >= topk) thr = cand;
    }
    int c = 0;
#pragma unroll
    for (int u = 0; u < KR; ++u) c += (kr[u] >= thr);
    exact = thr != 0u && __ballot_sync(kFull, c > 4) == 0u;
    nge = c;
  }
  if (!exact) {
    // bitwise search over all keys, from the highest bit in which the row's candidates differ
    uint32_t kmin = 0xffffffffu;
#pragma unroll
    for (int u = 0; u < KR; ++u)
      if (in_range(lane + 32 * u)) kmin = min(kmin, kr[u]);
    kmin = __reduce_min_sync(kFull, kmin);
    const int top_bit = 31 - __clz(kmin ^ kmaxv);
    thr = (top_bit >= 31) ? 0u : (kmaxv & ~((2u << max(top_bit, 0)) - 1u));
    if (top_bit < 0) thr = kmaxv;
    for (int bit = top_bit; bit >= 0; --bit) {
      const uint32_t cand = thr | (1u << bit);
      int cnt = 0;
#pragma unroll
      for (int u = 0; u < KR; ++u) cnt += (kr[u] >= cand);
      cnt = __reduce_add_sync(kFull, cnt);
      if (cnt >= topk) thr = cand;
    }
    nge = 0;
#pragma unroll
    for (int u = 0; u < KR; ++u) nge += (kr[u] >= thr);
  }
  // ordered compaction: keys above the threshold, then the lowest-indexed keys equal to it.  With thr >= 1
  // the zero keys that stand for blocks outside the candidate range never pass a comparison (thr = 0 only
  // when a candidate's own key is 0, the key of one NaN pattern: the general path below handles it).
  nge = __reduce_add_sync(kFull, nge);
  const uint32_t lt_mask = (1u << lane) - 1u;
  int out = 0;
  if (nge == topk && thr != 0u) {   // no surplus of keys equal to the threshold: keep every key >= thr
#pragma unroll
    for (int u = 0; u < KR; ++u) {
      const uint32_t keep_ballot = __ballot_sync(kFull, kr[u] >= thr);
      if (keep_ballot != 0u) {
        if (kr[u] >= thr) dst[out + __popc(keep_ballot & lt_mask)] = lane + 32 * u;
        out += __popc(keep_ballot);
      }
    }
    return;
  }
  int ngreater = 0;
#pragma unroll
  for (int u = 0; u < KR; ++u) ngreater += (kr[u] > thr);
  ngreater = __reduce_add_sync(kFull, ngreater);
  const int ties_allowed = topk - ngreater;  // >= 1: lowest indices among the keys equal to thr
  int ties_seen = 0;
#pragma unroll
  for (int u = 0; u < KR; ++u) {
    if (32 * u < nb) {
      const int j = lane + 32 * u;
      const bool valid = in_range(j);
      const bool tie = valid && (kr[u] == thr);
      const uint32_t tie_ballot = __ballot_sync(kFull, tie);
      const int tie_rank = ties_seen + __popc(tie_ballot & lt_mask);
      const bool keep = valid && ((kr[u] > thr) || (tie && tie_rank < ties_allowed));
      const uint32_t keep_ballot = __ballot_sync(kFull, keep);
      if (keep) dst[out + __popc(keep_ballot & lt_mask)] = j;
      out += __popc(keep_ballot);
      ties_seen += __popc(tie_ballot);
    }
  }
}

template <int D, int ROWS, bool WINDOW>
__global__ void __launch_bounds__(kTopkThreads, ROWS == 16 ? 3 : 4)
topk_kernel(const float* __restrict__ pq, const float* __restrict__ pkT, int32_t* __restrict__ kept_idx,
            int32_t* __restrict__ kept_cnt, int nb, int nbp, int topk, int groups_per_bh, int N, int blk_size,
            int frame_tokens, int window) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // pooled Q of the CTA's ROWS query blocks, channel-major: s_pq[c][r], so that one 16-byte load
  // yields four rows of one channel as two packed fp32x2 operands
  float* s_pq = reinterpret_cast<float*>(smem_raw);                   // [D][ROWS]
  uint32_t* s_key = reinterpret_cast<uint32_t*>(s_pq + ROWS * D);     // [ROWS][nbp]

  const int64_t bh = blockIdx.x / groups_per_bh;
  const int i0 = (blockIdx.x % groups_per_bh) * ROWS;
  const int nrows = min(ROWS, nb - i0);

  for (int e = threadIdx.x; e < ROWS * D; e += kTopkThreads) {
    const int r = e / D, c = e % D;
    s_pq[c * ROWS + r] = (r < nrows) ? pq[(bh * nb + i0 + r) * D + c] : 0.0f;
  }
  __syncthreads();

  // scores: a thread owns 4 adjacent key blocks (one 16-byte load per channel) and walks the channels
  // in ascending order for the CTA's ROWS query blocks at once: a ROWS x 4 register tile.
  // fma.rn.f32x2 is a pair of IEEE fmaf over two rows, so every accumulator still sees exactly the
  // chain a = fmaf(pq[i,c], pk[j,c], a), c ascending.  Columns nb..nbp-1 of pooled K are padding
  // whose scores are stored but never read.
  const float* kcol = pkT + bh * D * (int64_t)nbp;
  const ulonglong2* s_pq2 = reinterpret_cast<const ulonglong2*>(s_pq);       // [D][ROWS / 4]
  constexpr int kPairs = ROWS / 2;
  constexpr int kCB = 4;   // channels per batch of loads; two batches (2 x 4 x 16 bytes) in flight per thread
  for (int j0 = threadIdx.x * 4; j0 < nb; j0 += kTopkThreads * 4) {
    uint64_t acc[4][kPairs];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int r = 0; r < kPairs; ++r) acc[u][r] = pack_f32x2(0.0f, 0.0f);
    const float* kp = kcol + j0;
    auto load_batch = [&](float4 (&kv)[kCB], int c0) {
#pragma unroll
      for (int cc = 0; cc < kCB; ++cc) kv[cc] = __ldg(reinterpret_cast<const float4*>(kp + (int64_t)(c0 + cc) * nbp));
    };
    auto fma_batch = [&](const float4 (&kv)[kCB], int c0) {
#pragma unroll
      for (int cc = 0; cc < kCB; ++cc) {
        uint64_t q2[kPairs];
#pragma unroll
        for (int g = 0; g < ROWS / 4; ++g) {
          const ulonglong2 t = s_pq2[(c0 + cc) * (ROWS / 4) + g];   // rows (4g, 4g+1), (4g+2, 4g+3)
          q2[2 * g] = t.x;
          q2[2 * g + 1] = t.y;
        }
        const uint64_t k2[4] = {pack_f32x2(kv[cc].x, kv[cc].x), pack_f32x2(kv[cc].y, kv[cc].y),
                                pack_f32x2(kv[cc].z, kv[cc].z), pack_f32x2(kv[cc].w, kv[cc].w)};
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int r = 0; r < kPairs; ++r) acc[u][r] = ffma2(q2[r], k2[u], acc[u][r]);
      }
    };
    float4 kva[kCB], kvb[kCB];
    load_batch(kva, 0);
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 2 * kCB) {
      load_batch(kvb, c0 + kCB);
      fma_batch(kva, c0);
      if (c0 + 2 * kCB < D) load_batch(kva, c0 + 2 * kCB);
      fma_batch(kvb, c0 + kCB);
    }
#pragma unroll
    for (int r = 0; r < kPairs; ++r) {
      uint4 lo, hi;
      float2 a;
      a = unpack_f32x2(acc[0][r]); lo.x = score_key(a.x); hi.x = score_key(a.y);
      a = unpack_f32x2(acc[1][r]); lo.y = score_key(a.x); hi.y = score_key(a.y);
      a = unpack_f32x2(acc[2][r]); lo.z = score_key(a.x); hi.z = score_key(a.y);
      a = unpack_f32x2(acc[3][r]); lo.w = score_key(a.x); hi.w = score_key(a.y);
      *reinterpret_cast<uint4*>(s_key + (2 * r) * nbp + j0) = lo;
      *reinterpret_cast<uint4*>(s_key + (2 * r + 1) * nbp + j0) = hi;
    }
  }
  __syncthreads();

  // selection: the CTA's warps take the rows round-robin, one warp per row
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int row = warp; row < nrows; row += kTopkThreads / 32) {
    const uint32_t* key = s_key + row * nbp;
    int32_t* dst = kept_idx + (bh * nb + i0 + row) * (int64_t)topk;
    // Causal frame window (Sec. 1, auto-regressive extension): only the key blocks that hold a key some
    // row of this query block may attend to are candidates, a contiguous run jlo..jhi.
    int jlo = 0, jhi = nb - 1;
    if constexpr (WINDOW) {
      const int r0 = (i0 + row) * blk_size, r1 = min((i0 + row + 1) * blk_size, N) - 1;
      const int f0 = max(r0 / frame_tokens - window + 1, 0);
      const int kend = (int)min((long long)(r1 / frame_tokens + 1) * frame_tokens, (long long)N);
      jlo = (int)((long long)f0 * frame_tokens / blk_size);
      jhi = (kend - 1) / blk_size;
    }
    const int k_row = min(topk, jhi - jlo + 1);
    if (nb <= 32 * 8) {
      select_row_regs<8, WINDOW>(key, nb, jlo, jhi, k_row, lane, dst);
    } else if (nb <= 32 * 20) {
      select_row_regs<20, WINDOW>(key, nb, jlo, jhi, k_row, lane, dst);
    } else if (nb <= 32 * 40) {
      select_row_regs<40, WINDOW>(key, nb, jlo, jhi, k_row, lane, dst);
    } else {
      select_row([&](int j) { return (WINDOW ? (j >= jlo && j <= jhi) : (j < nb)) ? key[j] : 0u; }, nb, jlo, jhi, k_row,
                 lane, dst);
    }
    if constexpr (WINDOW)
      for (int t = k_row + lane; t < topk; t += 32) dst[t] = -1;    // unused tail of a list cut short by the window
    if (lane == 0 && kept_cnt != nullptr) kept_cnt[bh * nb + i0 + row] = k_row;
  }
}

template <int D, int ROWS>
static int launch_topk(const float* pq, const float* pkT, int32_t* kept_idx, int32_t* kept_cnt, int nb, int nbp, int topk,
                       int64_t bh, int N, int block, int frame_tokens, int window, cudaStream_t stream) {
  const int groups = (nb + ROWS - 1) / ROWS;
  const int64_t ctas = bh * groups;
  if (ctas > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const size_t smem = (size_t)ROWS * D * sizeof(float) + (size_t)ROWS * nbp * sizeof(uint32_t);
  auto kern = frame_tokens > 0 ? topk_kernel<D, ROWS, true> : topk_kernel<D, ROWS, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return SPARKATTN_E_CUDA;
  kern<<<(unsigned)ctas, kTopkThreads, smem, stream>>>(pq, pkT, kept_idx, kept_cnt, nb, nbp, topk, groups, N, block,
                                                       frame_tokens, window);
  return SPARKATTN_OK;
}

// Where the pooled means live in a selection workspace: pooled Q [B*H][nb][d] right behind the header, pooled K
// transposed [B*H][d][nbp] behind it.
float* select_pooled_ptr(const sparkattn_shape_t& s, void* workspace, bool key_side) {
  const int nb = (s.N + s.block - 1) / s.block;
  float* pq = reinterpret_cast<float*>(static_cast<char*>(workspace) + kWorkspaceHeaderBytes);
  return key_side ? pq + (int64_t)s.B * s.H * nb * s.d : pq;
}

// scores + top-k on pooled means that are already in the workspace
static int launch_topk_any(const sparkattn_shape_t& s, int topk, int frame_tokens, int window, int32_t* kept_idx,
                           int32_t* kept_cnt, void* workspace, cudaStream_t stream) {
  const int nb = (s.N + s.block - 1) / s.block;
  const int nbp = round_up(nb, 32);
  const int64_t bh = (int64_t)s.B * s.H;
  const float* pq = select_pooled_ptr(s, workspace, false);
  const float* pkT = select_pooled_ptr(s, workspace, true);
  // 16 query blocks per CTA while two CTAs' score rows fit one SM's shared memory and the grid still
  // fills the device several times over (small problems are bound by the latency of one CTA), else 8
  constexpr int kNumSMs = 148;   // B200; another count only moves the point where the CTAs get smaller
  const bool rows16 = (size_t)16 * nbp * sizeof(uint32_t) <= 100u * 1024u && bh * ((nb + 15) / 16) >= 6 * kNumSMs;
  if (s.d == 128)
    return rows16 ? launch_topk<128, 16>(pq, pkT, kept_idx, kept_cnt, nb, nbp, topk, bh, s.N, s.block, frame_tokens, window, stream)
                  : launch_topk<128, 8>(pq, pkT, kept_idx, kept_cnt, nb, nbp, topk, bh, s.N, s.block, frame_tokens, window, stream);
  if (s.d == 64)
    return rows16 ? launch_topk<64, 16>(pq, pkT, kept_idx, kept_cnt, nb, nbp, topk, bh, s.N, s.block, frame_tokens, window, stream)
                  : launch_topk<64, 8>(pq, pkT, kept_idx, kept_cnt, nb, nbp, topk, bh, s.N, s.block, frame_tokens, window, stream);
  return SPARKATTN_E_UNSUPPORTED_SHAPE;
}

int launch_select_pooled(const sparkattn_shape_t& s, int topk, int32_t* kept_idx, int32_t* kept_cnt, void* workspace,
                         cudaStream_t stream) {
  const int nb = (s.N + s.block - 1) / s.block;
  if (nb > kSelectMaxBlocks) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const int rc = launch_topk_any(s, topk, 0, 0, kept_idx, kept_cnt, workspace, stream);
  if (rc != SPARKATTN_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

int launch_select(const sparkattn_shape_t& s, const void* q, const void* k, int topk, int frame_tokens, int window,
                  const int32_t* block_valid, int32_t* kept_idx, int32_t* kept_cnt, void* workspace, cudaStream_t stream) {
  const int nb = (s.N + s.block - 1) / s.block;
  const int nbp = round_up(nb, 32);
  if (nb > kSelectMaxBlocks) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const int64_t n_items = (int64_t)s.B * s.H * nb;
  float* pq = select_pooled_ptr(s, workspace, false);
  float* pkT = select_pooled_ptr(s, workspace, true);
  const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
  const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
  const int64_t pool_ctas = (2 * n_items + kPoolThreads / 32 - 1) / (kPoolThreads / 32);
  if (pool_ctas > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (s.d == 128) {
    pool_kernel<128><<<(unsigned)pool_ctas, kPoolThreads, 0, stream>>>(
        qb, kb, pq, pkT, s.H, s.N, s.block, nb, nbp, s.stride_b, s.stride_h, s.stride_n, n_items, block_valid);
  } else if (s.d == 64) {
    pool_kernel<64><<<(unsigned)pool_ctas, kPoolThreads, 0, stream>>>(
        qb, kb, pq, pkT, s.H, s.N, s.block, nb, nbp, s.stride_b, s.stride_h, s.stride_n, n_items, block_valid);
  } else {
    return SPARKATTN_E_UNSUPPORTED_SHAPE;
  }
  const int rc = launch_topk_any(s, topk, frame_tokens, window, kept_idx, kept_cnt, workspace, stream);
  if (rc != SPARKATTN_OK) return rc;
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

}  // namespace sparkattn
