// Low-rank compensation branch and gate fusion of the paper's attention module (Sec. 4.1):
//   q~_i = R_r(p_i) silu(P_q q_i),  k~_j = R_r(p_j) silu(P_k k_j),  C = sum_j k~_j v_j^T,
//   O_lr,i = RMSNorm(q~_i^T C),  O_i = O_s,i + g_i r_i O_lr,i,  r_i = RMS(O_s,i).
// Linear in the sequence length; both passes are streaming and HBM-bound, their contractions
// (projection to rank r = 64, k~ v^T accumulation, q~ C) run as tcgen05 MMAs with TMEM accumulators.
//
// Both kernels run one CTA per SM over a contiguous chunk of 128-token tiles of one (batch, head),
// with three feature warpgroups that take the tiles round-robin (a thread owns one token row), one
// TMA producer warp and one MMA-issuing warp:
//   comp_state_kernel   per tile: T = K P_k^T (MMA) -> silu + rotary on the T rows -> k~ as bf16
//                       into shared memory -> C^T += V^T k~ (MMA, both operands MN-major straight
//                       from the row-major tiles).  The chunk's C^T goes to the workspace;
//                       comp_reduce_kernel adds the chunks in a fixed order.
//   comp_apply_kernel   per tile: T = Q P_q^T -> silu + rotary -> q~ (bf16, shared memory) ->
//                       Y = q~ C (MMA, C as bf16 in shared memory; Y overwrites T in TMEM) ->
//                       per row RMSNorm, RMS of the sparse output row (a TMA tile in the slot the
//                       Q tile used), gate, add in place, TMA store.
// The MMA warp polls for whichever product is ready next (projection of a new tile, or the second
// product of the oldest tile whose features are written), so the three warpgroups, the loads and
// the tensor pipe overlap.  Every wait is bounded; rows past N are zero tiles (TMA fill) and are
// never stored.
#include <cuda.h>

#include "common.cuh"
#include "launch.h"
#include "rope.cuh"
#include "tmap.h"

namespace sparkattn {

constexpr int kFeatWGs = 3;
constexpr int kCompThreads = kFeatWGs * 128 + 128;  // feature warpgroups, then a warpgroup holding the TMA warp and the MMA warp
constexpr int kFeatRegs = 152, kCtrlRegs = 56;      // register split between the two kinds of warpgroup
constexpr int kProducerWarp = kFeatWGs * 4;
constexpr int kMmaWarp = kFeatWGs * 4 + 1;
constexpr int kRank = 64;
constexpr int kCD = 128;              // head dimension handled by this file
constexpr int kTileTok = 128;
constexpr int kNumSMs = 148;          // chunking target (B200); any other count only changes the balance

struct CompParams {
  RopeTable rope;
  int H, N, nt;                       // nt = number of 128-token tiles
  int tiles_per_cta, nchunks;
  int64_t stride_b, stride_h, stride_n;
  float* partial;                     // state: [BH][nchunks][d][r] fp32
  const float* state;                 // apply: [BH][r][d] fp32
  const float* gate;                  // apply: [BH][N]
  const __nv_bfloat16* o_sparse;      // apply
  __nv_bfloat16* out;                 // apply
  float eps;
  const float2* rope_table;           // [T + Hg + Wg][rank/2] (cos, sin)
  int32_t* status;
};

// cos/sin of every (coordinate, rotary pair) the grid can produce, position-major so that a token's
// pairs of one axis sit in one 256-byte row: table[(base(axis) + e) * 32 + m] = (cos, sin)(e * freq[m])
// with base(t) = 0, base(y) = T, base(x) = T + Hg (entries of pairs that rotate by another axis are
// unused).  A few thousand entries; the feature loops read it through L1 instead of running a
// full-range sincosf per (token, pair).
__global__ void rope_table_kernel(const RopeTable rope, float2* __restrict__ table) {
  const int m = threadIdx.x;                         // rank/2 threads
  const int ax = rope.axis[m];
  const int e = blockIdx.x;                          // T + Hg + Wg blocks
  const int lo = ax == 0 ? 0 : (ax == 1 ? rope.T : rope.T + rope.Hg);
  const int hi = ax == 0 ? rope.T : (ax == 1 ? rope.T + rope.Hg : rope.T + rope.Hg + rope.Wg);
  float sn = 0.0f, cs = 1.0f;
  if (e >= lo && e < hi) sincosf((float)(e - lo) * rope.freq[m], &sn, &cs);
  table[e * (kRank / 2) + m] = make_float2(cs, sn);
}

__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// The (cos, sin) pairs of one token's rank/2 feature pairs, requested from the position-major table.  Called
// before the wait for the token tile's projection, so that the table's L2 latency is not on the row's path.
__device__ __forceinline__ void rope_factors(float2 (&cs)[kRank / 2], const RopeTable& rope,
                                             const float2* __restrict__ table, int token) {
  const int x = token % rope.Wg;
  const int yy = token / rope.Wg;
  const int y = yy % rope.Hg;
  const int t = yy / rope.Hg;
  const float2* row_t = table + t * (kRank / 2);
  const float2* row_y = table + (rope.T + y) * (kRank / 2);
  const float2* row_x = table + (rope.T + rope.Hg + x) * (kRank / 2);
#pragma unroll
  for (int m = 0; m < kRank / 2; ++m) {
    const int ax = rope.axis[m];
    cs[m] = __ldg((ax == 0 ? row_t : (ax == 1 ? row_y : row_x)) + m);
  }
}

// One token row of T (64 fp32 columns at `taddr`) -> silu -> rank-truncated rotary rotation of the
// adjacent pairs -> bf16 -> row `row` of a [128 rows x 128 B] tile with 128-byte swizzle.
// Done in two halves of 32 columns to bound the live registers.
__device__ __forceinline__ void feature_row(uint32_t taddr, unsigned char* tile, int row, const float2 (&cs)[kRank / 2]) {
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    uint32_t r[32];
    tmem_ld32(taddr + half * 32, r);
    tc_wait_ld();
    uint32_t w[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float2 cj = cs[half * 16 + j];
      const float u0 = __uint_as_float(r[2 * j]), u1 = __uint_as_float(r[2 * j + 1]);
      const float2 e = unpack_f32x2(fadd2(pack_f32x2(fast_exp2(u0 * -1.4426950408889634f), fast_exp2(u1 * -1.4426950408889634f)),
                                          pack_f32x2(1.0f, 1.0f)));
      const float z0 = u0 * fast_rcp(e.x), z1 = u1 * fast_rcp(e.y);
      const float o0 = fmaf(z0, cj.x, -z1 * cj.y);
      const float o1 = fmaf(z0, cj.y, z1 * cj.x);
      const __nv_bfloat162 h2 = __floats2bfloat162_rn(o0, o1);
      w[j] = *reinterpret_cast<const uint32_t*>(&h2);
    }
#pragma unroll
    for (int c = 0; c < 4; ++c)
      *reinterpret_cast<uint4*>(tile + row * 128 + (((half * 4 + c) ^ (row & 7)) << 4)) =
          make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
  }
}

// instruction descriptor with both major bits explicit (bf16 in, fp32 accumulate)
__host__ __device__ constexpr uint32_t comp_idesc(uint32_t M, uint32_t N, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) | ((N >> 3) << 17) |
         ((M >> 4) << 24);
}

// T[128 tokens x 64] = X[128 x 128] P^T : X tile K-major (2 slabs of 16 KB), P K-major (2 slabs of 8 KB)
__device__ __forceinline__ void issue_projection(uint32_t tmem_T, uint32_t x_smem, uint32_t p_smem) {
  const uint64_t dX = make_smem_desc_sw128(x_smem, 16), dP = make_smem_desc_sw128(p_smem, 16);
  const uint32_t x_lo = (uint32_t)dX, x_hi = (uint32_t)(dX >> 32), p_lo = (uint32_t)dP, p_hi = (uint32_t)(dP >> 32);
  constexpr uint32_t idesc = comp_idesc(128, kRank, false, false);
#pragma unroll
  for (int s = 0; s < 2; ++s)
#pragma unroll
    for (int kk = 0; kk < 4; ++kk)
      mma_ss<false>(tmem_T, make_desc(x_lo + ((s * 16384 + kk * 32) >> 4), x_hi),
                    make_desc(p_lo + ((s * 8192 + kk * 32) >> 4), p_hi), idesc, (s | kk) != 0 ? 1u : 0u);
}

// Idle bookkeeping of the polling MMA warp: false once the CTA was aborted or nothing became ready
// for kWaitLimitNs.
struct IdleGuard {
  uint64_t t0;
  uint32_t polls;
  __device__ __forceinline__ void reset() { polls = 0; }
  __device__ __forceinline__ bool idle(volatile int* abort_flag, int32_t* status, int wait_id) {
    if (polls == 0) t0 = global_timer_ns();
    if ((++polls & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        report_status(status, SPARKATTN_E_DEVICE_TIMEOUT, wait_id);
        return false;
      }
    }
    return true;
  }
};

// state kernel shared memory: P | K ring (2) | V ring (2) | k~ tiles (one per warpgroup) | barriers
constexpr int kStateOffK = 16384, kStateOffV = kStateOffK + 2 * 32768, kStateOffF = kStateOffV + 2 * 32768;
constexpr int kStateOffBar = kStateOffF + kFeatWGs * 16384;
constexpr int kStateSmem = 1024 + kStateOffBar + 256;
// apply kernel shared memory: P | C | Q ring (3) | q~ tiles | barriers
constexpr int kApplyOffC = 16384, kApplyOffQ = 32768, kApplyOffF = kApplyOffQ + kFeatWGs * 32768;
constexpr int kApplyOffBar = kApplyOffF + kFeatWGs * 16384;
constexpr int kApplySmem = 1024 + kApplyOffBar + 256;

__global__ void __launch_bounds__(kCompThreads, 1)
comp_state_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                  const __grid_constant__ CUtensorMap tmap_p, const CompParams p) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* sP = smem;
  unsigned char* sK = smem + kStateOffK;
  unsigned char* sV = smem + kStateOffV;
  unsigned char* sF = smem + kStateOffF;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStateOffBar);
  uint64_t* bar_p_full = bars + 0;
  uint64_t* bar_k_full = bars + 1;    // [2] TMA landed
  uint64_t* bar_k_empty = bars + 3;   // [2] projection MMAs done
  uint64_t* bar_v_full = bars + 5;    // [2]
  uint64_t* bar_v_empty = bars + 7;   // [2] accumulation MMAs done
  uint64_t* bar_t_full = bars + 9;    // [3] projection of a tile in T[g]
  uint64_t* bar_f_full = bars + 12;   // [3] k~ tile g written (128 arrivals)
  uint64_t* bar_f_empty = bars + 15;  // [3] accumulation MMAs that read k~ tile g done
  uint64_t* bar_acc = bars + 18;      // everything issued is complete
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 20);
  volatile int* s_abort = reinterpret_cast<volatile int*>(bars + 21);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, bh = blockIdx.y;
  const int h = bh % p.H, b = bh / p.H;
  const int tile0 = chunk * p.tiles_per_cta;
  const int ntiles = max(0, min(p.tiles_per_cta, p.nt - tile0));

  if (threadIdx.x == 0) {
    mbar_init(bar_p_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_k_full + i, 1); mbar_init(bar_k_empty + i, 1);
      mbar_init(bar_v_full + i, 1); mbar_init(bar_v_empty + i, 1);
    }
    for (int g = 0; g < kFeatWGs; ++g) {
      mbar_init(bar_t_full + g, 1); mbar_init(bar_f_full + g, 128); mbar_init(bar_f_empty + g, 1);
    }
    mbar_init(bar_acc, 1);
    *s_abort = 0;
    mbar_fence_init();
  }
  if (warp == kProducerWarp) {
    tmem_alloc(s_tmem, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const uint32_t tmem_C = tmem + kFeatWGs * 64;    // T[g] at column 64 g, C^T behind them

  if (warp >= kProducerWarp) reg_dec<kCtrlRegs>();
  if (warp == kProducerWarp) {
    if (lane == 0 && ntiles > 0) {
      mbar_expect_tx(bar_p_full, 16384);
      tma_load_4d(sP, &tmap_p, bar_p_full, 0, 0, h, 0);
      tma_load_4d(sP + 8192, &tmap_p, bar_p_full, 64, 0, h, 0);
      int ik = 0, iv = 0;                          // next K tile / next V tile to request
      bool ok = true;
      IdleGuard guard;
      guard.reset();
      while (ok && iv < ntiles) {
        bool progressed = false;
        if (ik < ntiles && (ik < 2 || mbar_try_wait(bar_k_empty + (ik & 1), ((ik >> 1) - 1) & 1))) {
          const int row = (tile0 + ik) * kTileTok, st = ik & 1;
          mbar_expect_tx(bar_k_full + st, 32768);
          tma_load_4d(sK + st * 32768, &tmap_k, bar_k_full + st, 0, row, h, b);
          tma_load_4d(sK + st * 32768 + 16384, &tmap_k, bar_k_full + st, 64, row, h, b);
          ++ik;
          progressed = true;
        }
        if (iv < 2 || mbar_try_wait(bar_v_empty + (iv & 1), ((iv >> 1) - 1) & 1)) {
          const int row = (tile0 + iv) * kTileTok, st = iv & 1;
          mbar_expect_tx(bar_v_full + st, 32768);
          tma_load_4d(sV + st * 32768, &tmap_v, bar_v_full + st, 0, row, h, b);
          tma_load_4d(sV + st * 32768 + 16384, &tmap_v, bar_v_full + st, 64, row, h, b);
          ++iv;
          progressed = true;
        }
        if (progressed) guard.reset();
        else ok = guard.idle(s_abort, p.status, 50);
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0 && ntiles > 0) {
      // C^T[128 d x 64 r] += V^T k~ : A = V tile (MN-major: d contiguous, two 64-column slabs),
      // B = k~ tile (MN-major: r contiguous), 16 tokens per MMA
      constexpr uint32_t idesc_acc = comp_idesc(128, kRank, true, true);
      bool ok = mbar_wait(bar_p_full, 0, s_abort, p.status, 52);
      int s1 = 0, s2 = 0;              // next tile to project / to accumulate
      IdleGuard guard;
      guard.reset();
      while (ok && s2 < ntiles) {
        bool progressed = false;
        // T[s1 % 3] is free once the features of tile s1 - 3 were consumed, i.e. s2 > s1 - 3
        if (s1 < ntiles && s1 - s2 < kFeatWGs && mbar_try_wait(bar_k_full + (s1 & 1), (s1 >> 1) & 1)) {
          tc_fence_after();
          issue_projection(tmem + (s1 % kFeatWGs) * 64, smem_u32(sK + (s1 & 1) * 32768), smem_u32(sP));
          tc_commit(bar_t_full + s1 % kFeatWGs);
          tc_commit(bar_k_empty + (s1 & 1));
          ++s1;
          progressed = true;
        }
        if (s2 < s1 && mbar_try_wait(bar_f_full + s2 % kFeatWGs, (s2 / kFeatWGs) & 1) &&
            mbar_try_wait(bar_v_full + (s2 & 1), (s2 >> 1) & 1)) {
          tc_fence_after();
          const uint64_t dV = make_smem_desc_sw128(smem_u32(sV + (s2 & 1) * 32768), 16384);
          const uint64_t dF = make_smem_desc_sw128(smem_u32(sF + (s2 % kFeatWGs) * 16384), 16);
          const uint32_t v_lo = (uint32_t)dV, v_hi = (uint32_t)(dV >> 32), f_lo = (uint32_t)dF, f_hi = (uint32_t)(dF >> 32);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            mma_ss<false>(tmem_C, make_desc(v_lo + ((kk * 2048) >> 4), v_hi), make_desc(f_lo + ((kk * 2048) >> 4), f_hi),
                          idesc_acc, (s2 | kk) != 0 ? 1u : 0u);
          tc_commit(bar_v_empty + (s2 & 1));
          tc_commit(bar_f_empty + s2 % kFeatWGs);
          ++s2;
          progressed = true;
        }
        if (progressed) guard.reset();
        else ok = guard.idle(s_abort, p.status, 53);
      }
      if (ok) tc_commit(bar_acc);
    }
  } else if (warp < kProducerWarp) {
    reg_inc<kFeatRegs>();
    const int g = warp >> 2;                              // warpgroup = tile slot
    const int row = threadIdx.x & 127;                    // token row of the tile = TMEM lane
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    unsigned char* tileF = sF + g * 16384;
    bool ok = true;
    for (int i = g, u = 0; ok && i < ntiles; i += kFeatWGs, ++u) {
      float2 cs[kRank / 2];
      rope_factors(cs, p.rope, p.rope_table, min((tile0 + i) * kTileTok + row, p.N - 1));   // rows past N are zero anyway
      ok = __all_sync(0xffffffffu, mbar_wait(bar_t_full + g, u & 1, s_abort, p.status, 56));
      if (!ok) break;
      if (u > 0) {                                        // k~ tile g still read by the previous accumulation?
        ok = __all_sync(0xffffffffu, mbar_wait(bar_f_empty + g, (u - 1) & 1, s_abort, p.status, 57));
        if (!ok) break;
      }
      tc_fence_after();
      feature_row(tmem + g * 64 + lane_off, tileF, row, cs);
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(bar_f_full + g);
    }
    if (g == 0) {
      float* dst = p.partial + (((int64_t)bh * p.nchunks + chunk) * kCD + row) * kRank;
      if (ntiles == 0) {
#pragma unroll
        for (int j = 0; j < 16; ++j) reinterpret_cast<uint4*>(dst)[j] = make_uint4(0u, 0u, 0u, 0u);
      } else if (ok && __all_sync(0xffffffffu, mbar_wait(bar_acc, 0, s_abort, p.status, 58))) {
        tc_fence_after();
        // thread = channel c of d; its TMEM row holds C^T[c][0..63]
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
          tmem_ld32(tmem_C + lane_off + half * 32, r);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 8; ++j)
            reinterpret_cast<uint4*>(dst + half * 32)[j] = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kProducerWarp) {
    if (*s_abort) __nanosleep(200000);
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

// state[bh][r][d] = sum over chunks (ascending) of partial[bh][chunk][d][r]
__global__ void comp_reduce_kernel(const float* __restrict__ partial, float* __restrict__ state, int nchunks) {
  const int bh = blockIdx.x;
  for (int e = threadIdx.x; e < kRank * kCD; e += blockDim.x) {
    const int a = e / kCD, c = e % kCD;
    float acc = 0.0f;
    for (int k = 0; k < nchunks; ++k) acc += partial[(((int64_t)bh * nchunks + k) * kCD + c) * kRank + a];
    state[((int64_t)bh * kRank + a) * kCD + c] = acc;
  }
}

// TMA store of a [128 rows x 64 columns] bf16 slab from shared memory (rows past the tensor's end are clipped)
__device__ __forceinline__ void tma_store_4d(const void* tmap, const void* smem_src, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
      ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// A ring slot of the apply kernel lives through: Q tile (TMA) -> projection MMAs -> sparse-branch
// tile O_s (TMA into the same bytes) -> fused output written in place by the warpgroup -> TMA
// store -> free.  Slot = warpgroup = tile % 3, so all global traffic of the tile is bulk copies.
__global__ void __launch_bounds__(kCompThreads, 1)
comp_apply_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_p,
                  const __grid_constant__ CUtensorMap tmap_os, const __grid_constant__ CUtensorMap tmap_out,
                  const CompParams p) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* sP = smem;
  unsigned char* sC = smem + kApplyOffC;           // C as bf16, [64 r rows][128 d], two 64-column slabs of 8 KB
  unsigned char* sQ = smem + kApplyOffQ;           // ring of 3 slots (Q, then O_s / O), slot = tile % 3
  unsigned char* sF = smem + kApplyOffF;           // q~ tiles, one per warpgroup
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kApplyOffBar);
  uint64_t* bar_p_full = bars + 0;
  uint64_t* bar_c_full = bars + 1;                 // C staged (128 arrivals)
  uint64_t* bar_q_full = bars + 2;                 // [3] Q tile landed
  uint64_t* bar_q_empty = bars + 5;                // [3] projection MMAs done: slot may take O_s
  uint64_t* bar_os_full = bars + 8;                // [3] O_s tile landed
  uint64_t* bar_t_full = bars + 11;                // [3]
  uint64_t* bar_f_full = bars + 14;                // [3] q~ tile written (128 arrivals)
  uint64_t* bar_y_full = bars + 17;                // [3] Y = q~ C done
  uint64_t* bar_slot_free = bars + 20;             // [3] output store has read the slot; Y has been read
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* s_abort = reinterpret_cast<volatile int*>(bars + 25);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y;
  const int h = bh % p.H, b = bh / p.H;
  const int tile0 = blockIdx.x * p.tiles_per_cta;
  const int ntiles = max(0, min(p.tiles_per_cta, p.nt - tile0));

  if (threadIdx.x == 0) {
    mbar_init(bar_p_full, 1);
    mbar_init(bar_c_full, 128);
    for (int g = 0; g < kFeatWGs; ++g) {
      mbar_init(bar_q_full + g, 1); mbar_init(bar_q_empty + g, 1); mbar_init(bar_os_full + g, 1);
      mbar_init(bar_t_full + g, 1); mbar_init(bar_f_full + g, 128); mbar_init(bar_y_full + g, 1);
      mbar_init(bar_slot_free + g, 1);
    }
    *s_abort = 0;
    mbar_fence_init();
  }
  if (warp == kProducerWarp) {
    tmem_alloc(s_tmem, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;                   // warpgroup g: columns [128 g, 128 g + 128): T in the first 64, then Y over all

  if (warp >= kProducerWarp) reg_dec<kCtrlRegs>();
  if (warp == kProducerWarp) {
    if (lane == 0 && ntiles > 0) {
      mbar_expect_tx(bar_p_full, 16384);
      tma_load_4d(sP, &tmap_p, bar_p_full, 0, 0, h, 0);
      tma_load_4d(sP + 8192, &tmap_p, bar_p_full, 64, 0, h, 0);
      int iq = 0, io = 0;                          // next Q tile / next O_s tile to request
      bool ok = true;
      IdleGuard guard;
      guard.reset();
      while (ok && io < ntiles) {
        bool progressed = false;
        if (iq < ntiles) {
          const int g = iq % kFeatWGs, n = iq / kFeatWGs;
          if (n == 0 || mbar_try_wait(bar_slot_free + g, (n - 1) & 1)) {
            const int row = (tile0 + iq) * kTileTok;
            mbar_expect_tx(bar_q_full + g, 32768);
            tma_load_4d(sQ + g * 32768, &tmap_q, bar_q_full + g, 0, row, h, b);
            tma_load_4d(sQ + g * 32768 + 16384, &tmap_q, bar_q_full + g, 64, row, h, b);
            ++iq;
            progressed = true;
          }
        }
        if (io < iq) {
          const int g = io % kFeatWGs;
          if (mbar_try_wait(bar_q_empty + g, (io / kFeatWGs) & 1)) {
            const int row = (tile0 + io) * kTileTok;
            mbar_expect_tx(bar_os_full + g, 32768);
            tma_load_4d(sQ + g * 32768, &tmap_os, bar_os_full + g, 0, row, h, b);
            tma_load_4d(sQ + g * 32768 + 16384, &tmap_os, bar_os_full + g, 64, row, h, b);
            ++io;
            progressed = true;
          }
        }
        if (progressed) guard.reset();
        else ok = guard.idle(s_abort, p.status, 60);
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0 && ntiles > 0) {
      // Y[128 tokens x 128 d] = q~ C : A = q~ tile (K-major: r contiguous), B = C (MN-major: d contiguous, two slabs)
      const uint64_t dC = make_smem_desc_sw128(smem_u32(sC), 8192);
      const uint32_t c_lo = (uint32_t)dC, c_hi = (uint32_t)(dC >> 32);
      constexpr uint32_t idesc_y = comp_idesc(128, kCD, false, true);
      bool ok = mbar_wait(bar_p_full, 0, s_abort, p.status, 61) && mbar_wait(bar_c_full, 0, s_abort, p.status, 62);
      int s1 = 0, s2 = 0;
      IdleGuard guard;
      guard.reset();
      while (ok && s2 < ntiles) {
        bool progressed = false;
        const int g1 = s1 % kFeatWGs;
        // a landed Q tile implies its slot (and with it the TMEM columns of the warpgroup) was released
        if (s1 < ntiles && mbar_try_wait(bar_q_full + g1, (s1 / kFeatWGs) & 1)) {
          tc_fence_after();
          issue_projection(tmem + g1 * 128, smem_u32(sQ + g1 * 32768), smem_u32(sP));
          tc_commit(bar_t_full + g1);
          tc_commit(bar_q_empty + g1);
          ++s1;
          progressed = true;
        }
        const int g2 = s2 % kFeatWGs;
        if (s2 < s1 && mbar_try_wait(bar_f_full + g2, (s2 / kFeatWGs) & 1)) {
          tc_fence_after();
          const uint64_t dF = make_smem_desc_sw128(smem_u32(sF + g2 * 16384), 16);
          const uint32_t f_lo = (uint32_t)dF, f_hi = (uint32_t)(dF >> 32);
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            mma_ss<false>(tmem + g2 * 128, make_desc(f_lo + ((kk * 32) >> 4), f_hi),
                          make_desc(c_lo + ((kk * 2048) >> 4), c_hi), idesc_y, kk != 0 ? 1u : 0u);
          tc_commit(bar_y_full + g2);
          ++s2;
          progressed = true;
        }
        if (progressed) guard.reset();
        else ok = guard.idle(s_abort, p.status, 63);
      }
    }
  } else if (warp < kProducerWarp) {
    reg_inc<kFeatRegs>();
    const int g = warp >> 2;
    const int row = threadIdx.x & 127;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    unsigned char* tileF = sF + g * 16384;
    unsigned char* slot = sQ + g * 32768;
    const uint32_t tmem_g = tmem + g * 128 + lane_off;
    if (g == 0) {
      if (ntiles > 0) {
        // stage C: thread j converts row a = j/2, columns [64*(j%2), +64) of the fp32 state to bf16
        const int a = row >> 1, half = row & 1;
        const float* src = p.state + ((int64_t)bh * kRank + a) * kCD + half * 64;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const float4 lo = __ldg(reinterpret_cast<const float4*>(src + 8 * c));
          const float4 hi = __ldg(reinterpret_cast<const float4*>(src + 8 * c + 4));
          const __nv_bfloat162 h0 = __floats2bfloat162_rn(lo.x, lo.y), h1 = __floats2bfloat162_rn(lo.z, lo.w);
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(hi.x, hi.y), h3 = __floats2bfloat162_rn(hi.z, hi.w);
          *reinterpret_cast<uint4*>(sC + half * 8192 + a * 128 + ((c ^ (a & 7)) << 4)) =
              make_uint4(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1),
                         *reinterpret_cast<const uint32_t*>(&h2), *reinterpret_cast<const uint32_t*>(&h3));
        }
        fence_proxy_async_smem();
      }
      mbar_arrive(bar_c_full);
    }
    bool ok = true;
    for (int i = g, u = 0; ok && i < ntiles; i += kFeatWGs, ++u) {
      const int tile_row = (tile0 + i) * kTileTok;
      const int token = tile_row + row;
      float2 cs[kRank / 2];
      rope_factors(cs, p.rope, p.rope_table, min(token, p.N - 1));
      const float gte = token < p.N ? __ldg(p.gate + (int64_t)bh * p.N + token) : 0.0f;
      ok = __all_sync(0xffffffffu, mbar_wait(bar_t_full + g, u & 1, s_abort, p.status, 64));
      if (!ok) break;
      tc_fence_after();
      // the previous tile of this warpgroup has passed its Y wait, so the q~ tile is free
      feature_row(tmem_g, tileF, row, cs);
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(bar_f_full + g);

      // sum of squares of the sparse-branch row (rows past N are zero tiles)
      ok = __all_sync(0xffffffffu, mbar_wait(bar_os_full + g, u & 1, s_abort, p.status, 66));
      if (!ok) break;
      float so = 0.0f;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 q4 = *reinterpret_cast<const uint4*>(slot + (c >> 3) * 16384 + row * 128 + (((c & 7) ^ (row & 7)) << 4));
        const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&q4);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(h2[j]);
          so = fmaf(f.x, f.x, fmaf(f.y, f.y, so));
        }
      }
      ok = __all_sync(0xffffffffu, mbar_wait(bar_y_full + g, u & 1, s_abort, p.status, 65));
      if (!ok) break;
      tc_fence_after();
      // two passes over Y in TMEM: sum of squares, then the fused output written over O_s in the slot
      float ss = 0.0f;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tmem_ld32(tmem_g + ch * 32, r);
        tc_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) ss = fmaf(__uint_as_float(r[j]), __uint_as_float(r[j]), ss);
      }
      const float coef = gte * sqrtf(so * (1.0f / kCD)) * rsqrtf(ss * (1.0f / kCD) + p.eps);
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        tmem_ld32(tmem_g + ch * 32, r);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4* cell = reinterpret_cast<uint4*>(slot + (ch >> 1) * 16384 + row * 128 +
                                                 ((((ch & 1) * 4 + c) ^ (row & 7)) << 4));
          const uint4 q4 = *cell;
          const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&q4);
          uint32_t w[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 f = __bfloat1622float2(h2[j]);
            const __nv_bfloat162 o2 = __floats2bfloat162_rn(fmaf(coef, __uint_as_float(r[8 * c + 2 * j]), f.x),
                                                            fmaf(coef, __uint_as_float(r[8 * c + 2 * j + 1]), f.y));
            w[j] = *reinterpret_cast<const uint32_t*>(&o2);
          }
          *cell = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
      fence_proxy_async_smem();
      tc_fence_before();
      named_bar_sync(1 + g, 128);
      if (row == 0) {
        tma_store_4d(&tmap_out, slot, 0, tile_row, h, b);
        tma_store_4d(&tmap_out, slot + 16384, 64, tile_row, h, b);
        bulk_commit();
        bulk_wait_read0();
        mbar_arrive(bar_slot_free + g);
      }
    }
    if (row == 0) bulk_wait0();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kProducerWarp) {
    if (*s_abort) __nanosleep(200000);
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ------------------------------------------------------------------ host side
static int comp_map(CUtensorMap* map, const void* base, cuuint64_t d0, cuuint64_t d1, cuuint64_t d2, cuuint64_t d3,
                    cuuint64_t s1, cuuint64_t s2, cuuint64_t s3, cuuint32_t box_rows) {
  const uint64_t dims[4] = {d0, d1, d2, d3};
  const uint64_t strides[3] = {s1, s2, s3};
  return make_slab_map(map, base, 2, dims, strides, box_rows);
}

// Chunks of token tiles per (batch, head): CTAs = B*H*chunks should fill whole waves of one CTA per
// SM.  Takes the smallest wave count whose last wave is at least 90 % full (else the fullest).
static int comp_chunks(const sparkattn_shape_t& s) {
  const int nt = (s.N + kTileTok - 1) / kTileTok;
  const long long bh = (long long)s.B * s.H;
  int best = 1;
  double best_fill = 0.0;
  for (int waves = 1; waves <= 6; ++waves) {
    long long nch = (long long)kNumSMs * waves / bh;
    if (nch < 1) continue;
    if (nch > nt) nch = nt;
    const int tpc = (int)((nt + nch - 1) / nch);
    nch = (nt + tpc - 1) / tpc;
    const double fill = (double)(bh * nch) / ((double)kNumSMs * waves);
    if (fill > best_fill + 1e-9) { best_fill = fill; best = (int)nch; }
    if (fill >= 0.9) break;
  }
  return best;
}

void launch_rope_table(const RopeTable& rope, float2* table, cudaStream_t stream) {
  rope_table_kernel<<<(unsigned)(rope.T + rope.Hg + rope.Wg), kRank / 2, 0, stream>>>(rope, table);
}

size_t rope_table_bytes(const int32_t* grid) {
  return ((size_t)(kRank / 2) * ((size_t)grid[0] + grid[1] + grid[2]) * sizeof(float2) + 255) / 256 * 256;
}

size_t comp_workspace_bytes(const sparkattn_shape_t& s, const int32_t* grid, bool with_state) {
  size_t bytes = kWorkspaceHeaderBytes + rope_table_bytes(grid);
  if (with_state) bytes += (size_t)s.B * s.H * comp_chunks(s) * kCD * kRank * sizeof(float);
  return bytes;
}

// header | rotary table | (state pass only) per-chunk partial states
static int prepare_workspace(CompParams& prm, const int32_t* grid, void* workspace, cudaStream_t stream) {
  char* base = static_cast<char*>(workspace);
  prm.status = reinterpret_cast<int32_t*>(base);
  float2* table = reinterpret_cast<float2*>(base + kWorkspaceHeaderBytes);
  prm.rope_table = table;
  prm.partial = reinterpret_cast<float*>(base + kWorkspaceHeaderBytes + rope_table_bytes(grid));
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  rope_table_kernel<<<(unsigned)(grid[0] + grid[1] + grid[2]), kRank / 2, 0, stream>>>(prm.rope, table);
  return SPARKATTN_OK;
}

static void fill_rope(CompParams& prm, const int32_t* grid, const int32_t* axis, const float* freq) {
  for (int m = 0; m < kRank / 2; ++m) { prm.rope.axis[m] = axis[m]; prm.rope.freq[m] = freq[m]; }
  prm.rope.T = grid[0]; prm.rope.Hg = grid[1]; prm.rope.Wg = grid[2];
}

int launch_comp_state(const sparkattn_shape_t& s, const void* k, const void* v, const void* pk, const int32_t* grid,
                      const int32_t* axis, const float* freq, float* state, void* workspace, cudaStream_t stream) {
  CUtensorMap mk, mv, mp;
  int rc;
  if ((rc = comp_map(&mk, k, s.d, s.N, s.H, s.B, s.stride_n, s.stride_h, s.stride_b, kTileTok)) != SPARKATTN_OK) return rc;
  if ((rc = comp_map(&mv, v, s.d, s.N, s.H, s.B, s.stride_n, s.stride_h, s.stride_b, kTileTok)) != SPARKATTN_OK) return rc;
  if ((rc = comp_map(&mp, pk, kCD, kRank, s.H, 1, kCD, (cuuint64_t)kRank * kCD, (cuuint64_t)s.H * kRank * kCD, kRank)) != SPARKATTN_OK)
    return rc;
  CompParams prm{};
  fill_rope(prm, grid, axis, freq);
  prm.H = s.H; prm.N = s.N; prm.nt = (s.N + kTileTok - 1) / kTileTok;
  prm.nchunks = comp_chunks(s);
  prm.tiles_per_cta = (prm.nt + prm.nchunks - 1) / prm.nchunks;
  prm.stride_b = s.stride_b; prm.stride_h = s.stride_h; prm.stride_n = s.stride_n;
  if ((rc = prepare_workspace(prm, grid, workspace, stream)) != SPARKATTN_OK) return rc;
  if (cudaFuncSetAttribute(comp_state_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStateSmem) != cudaSuccess)
    return SPARKATTN_E_CUDA;
  const dim3 grid_dim((unsigned)prm.nchunks, (unsigned)(s.B * s.H));
  comp_state_kernel<<<grid_dim, kCompThreads, kStateSmem, stream>>>(mk, mv, mp, prm);
  comp_reduce_kernel<<<(unsigned)(s.B * s.H), 256, 0, stream>>>(prm.partial, state, prm.nchunks);
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

int launch_comp_apply(const sparkattn_shape_t& s, const void* q, const void* pq, const int32_t* grid,
                      const int32_t* axis, const float* freq, const float* state, const float* gate,
                      const void* o_sparse, void* out, float eps, void* workspace, cudaStream_t stream) {
  CUtensorMap mq, mp, mos, mout;
  int rc;
  if ((rc = comp_map(&mq, q, s.d, s.N, s.H, s.B, s.stride_n, s.stride_h, s.stride_b, kTileTok)) != SPARKATTN_OK) return rc;
  if ((rc = comp_map(&mos, o_sparse, s.d, s.N, s.H, s.B, s.stride_n, s.stride_h, s.stride_b, kTileTok)) != SPARKATTN_OK) return rc;
  if ((rc = comp_map(&mout, out, s.d, s.N, s.H, s.B, s.stride_n, s.stride_h, s.stride_b, kTileTok)) != SPARKATTN_OK) return rc;
  if ((rc = comp_map(&mp, pq, kCD, kRank, s.H, 1, kCD, (cuuint64_t)kRank * kCD, (cuuint64_t)s.H * kRank * kCD, kRank)) != SPARKATTN_OK)
    return rc;
  CompParams prm{};
  fill_rope(prm, grid, axis, freq);
  prm.H = s.H; prm.N = s.N; prm.nt = (s.N + kTileTok - 1) / kTileTok;
  prm.tiles_per_cta = (prm.nt + comp_chunks(s) - 1) / comp_chunks(s);
  prm.nchunks = (prm.nt + prm.tiles_per_cta - 1) / prm.tiles_per_cta;
  prm.stride_b = s.stride_b; prm.stride_h = s.stride_h; prm.stride_n = s.stride_n;
  prm.state = state; prm.gate = gate;
  prm.o_sparse = static_cast<const __nv_bfloat16*>(o_sparse);
  prm.out = static_cast<__nv_bfloat16*>(out);
  prm.eps = eps;
  if ((rc = prepare_workspace(prm, grid, workspace, stream)) != SPARKATTN_OK) return rc;
  if (cudaFuncSetAttribute(comp_apply_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kApplySmem) != cudaSuccess)
    return SPARKATTN_E_CUDA;
  const dim3 grid_dim((unsigned)prm.nchunks, (unsigned)(s.B * s.H));
  comp_apply_kernel<<<grid_dim, kCompThreads, kApplySmem, stream>>>(mq, mp, mos, mout, prm);
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

}  // namespace sparkattn
