// sparkattn_fwd: block-sparse flash-attention forward for sm_100a.
//
// Computes the paper's sparse branch O_s = A_M(Q, K, V) (Sec. 4.1): exact
// softmax attention (Sec. 2, softmax(Q K^T / sqrt(d)) V) restricted, for every
// query block, to the key blocks of its kept list.
//
// One CTA owns one (batch, head, query block) work item; two CTAs share an SM
// so that one item's softmax overlaps the other's tensor-core work.
//   warps 0-3  softmax: thread r owns query row r.  One tcgen05.ld pass brings
//              the whole S row into registers (this warpgroup raises its
//              register budget, the other lowers its own), fp32 online softmax
//              with packed fp32x2 FMA/ADD and 3-input max (row max / row sum
//              need no shuffles: a row lives in one thread), P written back to
//              TMEM over S in the input precision, conditional rescale of O,
//              final normalise and store.
//   warp 4     TMA producer: Q tile once, then K_j / V_j tiles of each kept
//              block into one K slot and one V slot (128-byte swizzle).
//   warp 5     MMA issuer: S = Q K_j^T (operands in shared memory) and
//              O += P V_j (P from TMEM, V MN-major from shared memory) as
//              tcgen05.mma with fp32 accumulators in TMEM.
//   warps 6-7  idle; they complete the second warpgroup so that it can hand
//              its registers to the softmax warpgroup.
// TMEM columns: [0, BLK) S (P overlays its first BLK*elt/4 columns), [BLK, BLK+D) O.
//
// Every wait on an mbarrier is bounded (common.cuh); a kept index outside
// [0, nb) is reported in the status word and its tile skipped by all roles.
#include <cuda.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "launch.h"
#include "tmap.h"

namespace sparkattn {

constexpr int kFwdThreads = 256;          // warps 0-3 softmax, 4 TMA, 5 MMA, 6-7 idle (fill the warpgroup)
constexpr int kSoftmaxRegs = 176;         // 128 * 176 + 128 * 80 = half of the SM's register file
constexpr int kOtherRegs = 80;
constexpr int kSoftmaxThreads = 128;
// In log2 units: O and l are only rescaled when the running row maximum grows
// by more than this; until then P may exceed 1 by at most 2^threshold, which
// bf16 holds without loss.  Exact: the final division by l uses the same
// reference maximum.  The FP8 path rescales on every increase (threshold 0)
// because its P is pre-scaled close to the E4M3 maximum.
constexpr float kLazyRescaleLog2 = 8.0f;
constexpr float kFp8PScaleLog2 = 8.0f;  // P * 2^8 <= 256 < 448

template <int D, int BLK, bool FP8>
struct FwdCfg {
  static constexpr int kElt = FP8 ? 1 : 2;
  static constexpr int kSlabs = D * kElt / 128;          // 128-byte-wide column slabs per tile
  static constexpr int kSlabElems = 128 / kElt;          // elements per slab row
  static constexpr int kQSlabBytes = 128 * 128;          // MMA M = 128 rows
  static constexpr int kKVSlabBytes = BLK * 128;
  static constexpr int kQBytes = kSlabs * kQSlabBytes;
  static constexpr int kKVBytes = kSlabs * kKVSlabBytes;
  static constexpr int kTileTxBytes = kSlabs * BLK * 128;  // bytes one Q / K / V load delivers
  static constexpr int kUmmaK = 32 / kElt;               // elements per MMA along K
  static constexpr int kQKSteps = 128 / 32;              // MMAs per slab for S
  static constexpr int kHalf = BLK / 2;                  // keys per pipeline step (half a key block)
  // S = Q K^T per half (N = BLK/2: lets S of the next tile start early, but each MMA is bound by
  // the shared-memory operand fetch) or per tile (N = BLK: full tensor rate).  Measured on B200:
  // the split wins when the MMAs are short (FP8), the full width when they are long (bf16).
  static constexpr bool kSplitS = FP8;
  static constexpr int kPVSteps = kHalf / kUmmaK;        // MMAs for O per half
  static constexpr int kListCap = kFwdMaxKept;           // kept-list entries staged in shared memory
  static constexpr int kTmemCols = (BLK + D) <= 128 ? 128 : 256;
  static constexpr int kSmemBytes = 1024 /*align slack*/ + kQBytes + 2 * kKVBytes + 256 /*barriers*/ + kListCap * 4;
  static_assert(D * kElt % 128 == 0 && BLK % 32 == 0 && D % 32 == 0, "tile shape");
};

struct FwdParams {
  const int32_t* kept_idx;
  const int32_t* kept_cnt;
  const float* q_scale;
  const float* k_scale;
  const float* v_scale;
  __nv_bfloat16* out;
  float* lse;
  int32_t* status;
  int H, N, nb, kmax;
  int frame_tokens, window;  // causal frame window (0 = none): key frame in (query frame - window, query frame]
  int64_t stride_b, stride_h, stride_n;
  float scale_log2;  // softmax_scale * log2(e)
};

template <int D, int BLK, bool FP8, bool WINDOW>
__global__ void __launch_bounds__(kFwdThreads, 2)
fwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
           const __grid_constant__ CUtensorMap tmap_v, const FwdParams p) {
  using Cfg = FwdCfg<D, BLK, FP8>;
  constexpr int HALF = Cfg::kHalf;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* sQ = smem;
  unsigned char* sK = sQ + Cfg::kQBytes;
  unsigned char* sV = sK + Cfg::kKVBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(sV + Cfg::kKVBytes);
  uint64_t* bar_q_full = bars + 0;
  uint64_t* bar_k_full = bars + 1;
  uint64_t* bar_v_full = bars + 2;
  uint64_t* bar_s_full = bars + 3;    // [2] S half complete (half 1 also: K slot free)
  uint64_t* bar_p_full = bars + 5;    // [2] P half written by all softmax threads
  uint64_t* bar_pv_done = bars + 7;   // [2] O += P_half V_half complete (half 1 also: V slot free)
  uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(bars + 10);
  volatile int* s_abort = reinterpret_cast<volatile int*>(bars + 11);
  int* s_ntiles = reinterpret_cast<int*>(bars + 12);
  int32_t* s_list = reinterpret_cast<int32_t*>(bars + 32);   // [kListCap] validated kept block indices

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int qb = blockIdx.x % p.nb;
  const int bh = blockIdx.x / p.nb;
  const int h = bh % p.H, b = bh / p.H;

  if (threadIdx.x == 0) {
    mbar_init(bar_q_full, 1);
    mbar_init(bar_k_full, 1);
    mbar_init(bar_v_full, 1);
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      mbar_init(bar_s_full + hf, 1);
      mbar_init(bar_p_full + hf, kSoftmaxThreads);
      mbar_init(bar_pv_done + hf, 1);
    }
    // a timeout recorded by an earlier CTA of this launch makes the rest of the grid drain at once
    *s_abort = (*reinterpret_cast<volatile int32_t*>(p.status) == SPARKATTN_E_DEVICE_TIMEOUT) ? 1 : 0;
    mbar_fence_init();
  }
  if (warp == 4) {
    if (lane == 0) {
      tma_prefetch_desc(&tmap_q);
      tma_prefetch_desc(&tmap_k);
      tma_prefetch_desc(&tmap_v);
    }
    __syncwarp();
    tmem_alloc(s_tmem_base, Cfg::kTmemCols);
    tmem_relinquish();
  } else if (warp == 6) {
    // Stage the kept list in shared memory, in order, dropping (and reporting) indices outside [0, nb).
    const int cnt = p.kept_cnt ? min(max(__ldg(p.kept_cnt + (int64_t)bh * p.nb + qb), 0), p.kmax) : p.kmax;
    const int32_t* list = p.kept_idx + ((int64_t)bh * p.nb + qb) * p.kmax;
    int out = 0;
    for (int base = 0; base < cnt; base += 32) {
      const int t = base + lane;
      const int kb = (t < cnt) ? __ldg(list + t) : 0;
      const bool valid = (t < cnt) && kb >= 0 && kb < p.nb;
      if (t < cnt && !valid) report_status(p.status, SPARKATTN_E_BAD_INDEX, kb);
      const uint32_t ballot = __ballot_sync(0xffffffffu, valid);
      if (valid) s_list[out + __popc(ballot & ((1u << lane) - 1u))] = kb;
      out += __popc(ballot);
    }
    if (lane == 0) *s_ntiles = out;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem_base;
  const uint32_t tmem_S = tmem;            // S half hf at columns [hf*HALF, (hf+1)*HALF); P half overlays its start
  const uint32_t tmem_O = tmem + BLK;
  const bool dead = *s_abort != 0;
  const int ntiles = *s_ntiles;

  if (warp >= 4) {
    reg_dec<kOtherRegs>();
  }
  if (dead) {
    // nothing to do: fall through to the teardown
  } else if (warp == 4) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      for (int n = 0; n < ntiles; ++n) {
        const int kb = s_list[n];
        if (n == 0) {
          mbar_expect_tx(bar_q_full, Cfg::kTileTxBytes);
#pragma unroll
          for (int s = 0; s < Cfg::kSlabs; ++s)
            tma_load_4d(sQ + s * Cfg::kQSlabBytes, &tmap_q, bar_q_full, s * Cfg::kSlabElems, qb * BLK, h, b);
        } else {
          if (!mbar_wait(bar_s_full + 1, (n - 1) & 1, s_abort, p.status, 1)) break;  // K slot free
        }
        mbar_expect_tx(bar_k_full, Cfg::kTileTxBytes);
#pragma unroll
        for (int s = 0; s < Cfg::kSlabs; ++s)
          tma_load_4d(sK + s * Cfg::kKVSlabBytes, &tmap_k, bar_k_full, s * Cfg::kSlabElems, kb * BLK, h, b);
        if (n > 0) {
          if (!mbar_wait(bar_pv_done + 1, (n - 1) & 1, s_abort, p.status, 2)) break;  // V slot free
        }
        mbar_expect_tx(bar_v_full, Cfg::kTileTxBytes);
#pragma unroll
        for (int s = 0; s < Cfg::kSlabs; ++s)
          tma_load_4d(sV + s * Cfg::kKVSlabBytes, &tmap_v, bar_v_full, s * Cfg::kSlabElems, kb * BLK, h, b);
      }
    }
  } else if (warp == 5) {
    // -------------------------------------------------------------- MMA issuer
    // Issue order (one thread; the tensor pipe executes in this order):
    //   split S:  S_0(0) S_1(0) | PV_0(n) S_0(n+1) PV_1(n) S_1(n+1) | ...
    //   full S:   S(0)          | PV_0(n) PV_1(n) S(n+1)            | ...
    // S(n+1) overwrites the columns P(n) lives in; it is issued right behind the PV that reads
    // them, and the softmax threads have finished reading S(n) before they signal P(n).
    if (lane == 0 && ntiles > 0) {
      constexpr uint32_t kFmt = FP8 ? 0u : 1u;
      constexpr bool kSplitS = Cfg::kSplitS;
      constexpr uint32_t idesc_qk = make_idesc(kFmt, 128, kSplitS ? HALF : BLK, false);
      constexpr uint32_t idesc_pv = make_idesc(kFmt, 128, D, true);
      // Descriptors are built once; per MMA only the 32-bit low word moves (start address in 16-byte
      // units), which keeps the single issuing thread far ahead of the tensor pipe.
      const uint64_t dQ = make_smem_desc_sw128(smem_u32(sQ), 16);
      const uint64_t dK = make_smem_desc_sw128(smem_u32(sK), 16);
      const uint64_t dV = make_smem_desc_sw128(smem_u32(sV), Cfg::kKVSlabBytes);
      const uint32_t q_lo = (uint32_t)dQ, q_hi = (uint32_t)(dQ >> 32);
      const uint32_t k_lo = (uint32_t)dK, k_hi = (uint32_t)(dK >> 32);
      const uint32_t v_lo = (uint32_t)dV, v_hi = (uint32_t)(dV >> 32);
      // S for half hf (split mode: N = HALF, one commit) or for the whole tile (N = BLK, hf = 0,
      // both halves' barriers signalled).
      auto issue_s = [&](int hf) {
        const uint32_t kh_lo = k_lo + ((hf * HALF * 128) >> 4);
#pragma unroll
        for (int s = 0; s < Cfg::kSlabs; ++s) {
#pragma unroll
          for (int kk = 0; kk < Cfg::kQKSteps; ++kk) {
            const uint64_t da = make_desc(q_lo + ((s * Cfg::kQSlabBytes + kk * 32) >> 4), q_hi);
            const uint64_t db = make_desc(kh_lo + ((s * Cfg::kKVSlabBytes + kk * 32) >> 4), k_hi);
            mma_ss<FP8>(tmem_S + hf * HALF, da, db, idesc_qk, (s | kk) != 0 ? 1u : 0u);
          }
        }
        tc_commit(bar_s_full + hf);
        if constexpr (!kSplitS) tc_commit(bar_s_full + 1);
      };
      auto issue_pv = [&](int hf, bool first) {
        const uint32_t vh_lo = v_lo + ((hf * HALF * 128) >> 4);
#pragma unroll
        for (int kk = 0; kk < Cfg::kPVSteps; ++kk) {
          const uint64_t db = make_desc(vh_lo + ((kk * Cfg::kUmmaK * 128) >> 4), v_hi);
          mma_ts<FP8>(tmem_O, tmem_S + hf * HALF + kk * 8, db, idesc_pv, (first && kk == 0) ? 0u : 1u);
        }
        tc_commit(bar_pv_done + hf);
      };
      bool ok = mbar_wait(bar_q_full, 0, s_abort, p.status, 3) && mbar_wait(bar_k_full, 0, s_abort, p.status, 5);
      if (ok) {
        tc_fence_after();
        issue_s(0);
        if constexpr (kSplitS) issue_s(1);
      }
      for (int n = 0; ok && n < ntiles; ++n) {
        const bool more = n + 1 < ntiles;
        if (!(ok = mbar_wait(bar_v_full, n & 1, s_abort, p.status, 6))) break;
        if (!(ok = mbar_wait(bar_p_full + 0, n & 1, s_abort, p.status, 7))) break;
        tc_fence_after();
        issue_pv(0, n == 0);
        if constexpr (kSplitS) {
          if (more) {
            if (!(ok = mbar_wait(bar_k_full, (n + 1) & 1, s_abort, p.status, 5))) break;
            tc_fence_after();
            issue_s(0);
          }
        }
        if (!(ok = mbar_wait(bar_p_full + 1, n & 1, s_abort, p.status, 7))) break;
        tc_fence_after();
        issue_pv(1, false);
        if (more) {
          if constexpr (kSplitS) {
            issue_s(1);
          } else {
            if (!(ok = mbar_wait(bar_k_full, (n + 1) & 1, s_abort, p.status, 5))) break;
            tc_fence_after();
            issue_s(0);
          }
        }
      }
    }
  } else if (warp < 4) {
    // ----------------------------------------------------------------- softmax
    reg_inc<kSoftmaxRegs>();
    const int row = threadIdx.x;                      // query row inside the block = TMEM lane
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    const int q_row = qb * BLK + row;
    const bool row_valid = row < BLK && q_row < p.N;
    // keys this row may attend to: [klo, khi) (everything up to N without a causal window)
    int klo = 0, khi = p.N;
    if constexpr (WINDOW) {
      const int fi = min(q_row, p.N - 1) / p.frame_tokens;
      klo = max(fi - p.window + 1, 0) * p.frame_tokens;
      khi = (int)min((long long)(fi + 1) * p.frame_tokens, (long long)p.N);
    }
    float m_used = 0.0f, l = 0.0f;
    float q_sc = 1.0f, v_max = 1.0f;
    if constexpr (FP8) {
      q_sc = __ldg(p.q_scale + (int64_t)bh * p.nb + qb);
      float vm = 0.0f;
      for (int j = 0; j < p.nb; ++j) vm = fmaxf(vm, __ldg(p.v_scale + (int64_t)bh * p.nb + j));
      v_max = vm;
    }
    bool ok = true;
    for (int n = 0; ok && n < ntiles; ++n) {
      const int kb = s_list[n];
      const int c_lo_tile = klo - kb * BLK, c_hi_tile = khi - kb * BLK;   // this row's valid columns of the tile
      float c = p.scale_log2;                        // logit -> log2 units
      float p_off = 0.0f;                            // log2 of the factor folded into P
      if constexpr (FP8) {
        c *= q_sc * __ldg(p.k_scale + (int64_t)bh * p.nb + kb);
        p_off = kFp8PScaleLog2 + log2f(__ldg(p.v_scale + (int64_t)bh * p.nb + kb) / v_max);
      }
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const int c_lo = c_lo_tile - hf * HALF, c_hi = c_hi_tile - hf * HALF;   // valid columns of this half: [c_lo, c_hi)
        ok = mbar_wait(bar_s_full + hf, n & 1, s_abort, p.status, 8);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();

        // this thread's half row of S, one pass over TMEM
        uint32_t sr[HALF];
#pragma unroll
        for (int ch = 0; ch < HALF / 32; ++ch)
          tmem_ld32(tmem_S + lane_off + hf * HALF + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[ch * 32]));
        tc_wait_ld();
        if ((WINDOW && c_lo > 0) || c_hi < HALF) {  // ragged last key block / keys outside the causal window get weight 0
#pragma unroll
          for (int i = 0; i < HALF; ++i)
            if ((WINDOW && i < c_lo) || i >= c_hi) sr[i] = 0xff800000u;
        }
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]);
        float mx2 = __uint_as_float(sr[2]), mx3 = __uint_as_float(sr[3]);
#pragma unroll
        for (int i = 4; i < HALF; i += 8) {
          mx0 = fmax3(mx0, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
          mx1 = fmax3(mx1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
          if (i + 4 < HALF) {
            mx2 = fmax3(mx2, __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
            mx3 = fmax3(mx3, __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
          }
        }
        const float m_new = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * c;
        float alpha = 1.0f;
        bool need = false;
        if ((n == 0 && hf == 0) || m_used == -INFINITY) {
          m_used = m_new;               // first half, or nothing accumulated for this row yet (all keys so far masked)
        } else if (m_new > m_used + (FP8 ? 0.0f : kLazyRescaleLog2)) {
          alpha = fast_exp2(m_used - m_new);
          m_used = m_new;
          need = true;
        }
        if (__any_sync(0xffffffffu, need)) {
          // O must be quiescent: the last PV issued before this point is the other half's
          // (previous tile's second half, or this tile's first half).
          const int prev_hf = hf ^ 1;
          const int prev_n = hf == 0 ? n - 1 : n;
          ok = mbar_wait(bar_pv_done + prev_hf, prev_n & 1, s_abort, p.status, 10);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after();
          l *= alpha;
          const uint64_t a2 = pack_f32x2(alpha, alpha);
#pragma unroll
          for (int ch = 0; ch < D / 32; ++ch) {
            uint32_t r[32];
            tmem_ld32(tmem_O + lane_off + ch * 32, r);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float2 o2 = unpack_f32x2(fmul2(pack_f32x2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), a2));
              r[i] = __float_as_uint(o2.x);
              r[i + 1] = __float_as_uint(o2.y);
            }
            tmem_st32(tmem_O + lane_off + ch * 32, r);
          }
        }

        // P = exp2(S*c - m) in the input precision, written over the start of this S half
        const float neg_m = m_used == -INFINITY ? 0.0f : p_off - m_used;   // a fully masked row: exp2(-inf) = 0, not NaN
        const uint64_t c2 = pack_f32x2(c, c), nm2 = pack_f32x2(neg_m, neg_m);
        uint64_t lsum0 = pack_f32x2(0.0f, 0.0f), lsum1 = lsum0;
        constexpr int kWordsPerChunk = FP8 ? 8 : 16;   // P words produced from 32 S columns
        constexpr int kHalfWords = HALF / 32 * kWordsPerChunk;
        uint32_t w[kHalfWords];
#pragma unroll
        for (int ch = 0; ch < HALF / 32; ++ch) {
          float e[32];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float2 x = unpack_f32x2(
                ffma2(pack_f32x2(__uint_as_float(sr[ch * 32 + i]), __uint_as_float(sr[ch * 32 + i + 1])), c2, nm2));
            e[i] = fast_exp2(x.x);
            e[i + 1] = fast_exp2(x.y);
            if ((i >> 1) & 1) lsum1 = fadd2(lsum1, pack_f32x2(e[i], e[i + 1]));
            else lsum0 = fadd2(lsum0, pack_f32x2(e[i], e[i + 1]));
          }
          if constexpr (FP8) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(e[4 * i], e[4 * i + 1]), __NV_SATFINITE, __NV_E4M3);
              const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(e[4 * i + 2], e[4 * i + 3]), __NV_SATFINITE, __NV_E4M3);
              w[ch * 8 + i] = lo | (hi << 16);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(e[2 * i], e[2 * i + 1]);
              w[ch * 16 + i] = *reinterpret_cast<const uint32_t*>(&h2);
            }
          }
        }
        static_assert(kHalfWords == 32 || kHalfWords == 16 || kHalfWords == 8, "P half width");
        if constexpr (kHalfWords == 32) tmem_st32(tmem_S + lane_off + hf * HALF, *reinterpret_cast<const uint32_t(*)[32]>(&w[0]));
        else if constexpr (kHalfWords == 16) tmem_st16(tmem_S + lane_off + hf * HALF, w);
        else tmem_st8(tmem_S + lane_off + hf * HALF, w);
        const float2 ls = unpack_f32x2(fadd2(lsum0, lsum1));
        const float l_tile = ls.x + ls.y;
        if constexpr (FP8) l += l_tile * fast_exp2(-p_off);
        else l += l_tile;
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_full + hf);
      }
    }

    // ---------------------------------------------------------------- epilogue
    __nv_bfloat16* orow = p.out + b * p.stride_b + h * p.stride_h + (int64_t)q_row * p.stride_n;
    if (ntiles == 0 || !ok) {
      if (row_valid && ok) {
#pragma unroll
        for (int ch = 0; ch < D / 8; ++ch) reinterpret_cast<uint4*>(orow)[ch] = make_uint4(0u, 0u, 0u, 0u);
        if (p.lse) p.lse[(int64_t)bh * p.N + q_row] = -INFINITY;
      }
    } else {
      ok = mbar_wait(bar_pv_done + 1, (ntiles - 1) & 1, s_abort, p.status, 9);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after();
        float inv = l > 0.0f ? 1.0f / l : 0.0f;     // no admissible key at all: zero row, lse = -inf
        if constexpr (FP8) inv *= v_max * fast_exp2(-kFp8PScaleLog2);
#pragma unroll
        for (int ch = 0; ch < D / 32; ++ch) {
          uint32_t r[32];
          tmem_ld32(tmem_O + lane_off + ch * 32, r);
          tc_wait_ld();
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint32_t ww[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[8 * i + 2 * j]) * inv,
                                                                __uint_as_float(r[8 * i + 2 * j + 1]) * inv);
                ww[j] = *reinterpret_cast<const uint32_t*>(&h2);
              }
              reinterpret_cast<uint4*>(orow + ch * 32)[i] = make_uint4(ww[0], ww[1], ww[2], ww[3]);
            }
          }
        }
        if (row_valid && p.lse) p.lse[(int64_t)bh * p.N + q_row] = (m_used + log2f(l)) * 0.6931471805599453f;
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    if (*s_abort) __nanosleep(200000);  // let copies / MMAs in flight land before the CTA's resources go
    tc_fence_after();
    tmem_dealloc(tmem, Cfg::kTmemCols);
  }
}

// ------------------------------------------------------------------ host side

size_t fwd_workspace_bytes(const sparkattn_shape_t& s, int kmax) {
  // the pipelined kernel keeps range-checked, compacted copies of the kept lists behind the header
  if (fwd_pipe_supported(s)) return fwd_pipe_workspace_bytes(s, kmax);
  return kWorkspaceHeaderBytes;
}

template <int D, int BLK, bool FP8>
static int launch_fwd_t(const sparkattn_shape_t& s, const CUtensorMap& mq, const CUtensorMap& mk,
                        const CUtensorMap& mv, const FwdParams& prm, cudaStream_t stream) {
  using Cfg = FwdCfg<D, BLK, FP8>;
  // at least 100 KB so that no more than two CTAs (2 x <=256 TMEM columns) share an SM
  const int smem = Cfg::kSmemBytes < 100 * 1024 ? 100 * 1024 : Cfg::kSmemBytes;
  auto kern = prm.frame_tokens > 0 ? fwd_kernel<D, BLK, FP8, true> : fwd_kernel<D, BLK, FP8, false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return SPARKATTN_E_CUDA;
  const long long ctas = (long long)s.B * s.H * prm.nb;
  if (ctas > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  kern<<<(unsigned)ctas, kFwdThreads, smem, stream>>>(mq, mk, mv, prm);
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

int launch_fwd(const sparkattn_shape_t& s, int dtype, const void* q, const void* k, const void* v,
               const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
               const int32_t* kept_cnt, int kmax, int frame_tokens, int window, const int32_t* block_valid, void* out,
               float* lse, void* workspace, cudaStream_t stream) {
  const bool fp8 = dtype == SPARKATTN_FP8_E4M3;
  if (fwd_pipe_supported(s))
    return launch_fwd_pipe(s, fp8, q, k, v, q_scale, k_scale, v_scale, kept_idx, kept_cnt, kmax, frame_tokens, window,
                           block_valid, out, lse, workspace, stream);
  // d = 128 always runs the persistent kernel; a sequence too long for its list pre-pass is not served
  if (s.d != 64 || s.block != 64 || fp8 || block_valid != nullptr) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  const int elt = fp8 ? 1 : 2;
  CUtensorMap mq, mk, mv;
  int rc;
  if ((rc = make_token_map(&mq, q, elt, s, s.block)) != SPARKATTN_OK) return rc;
  if ((rc = make_token_map(&mk, k, elt, s, s.block)) != SPARKATTN_OK) return rc;
  if ((rc = make_token_map(&mv, v, elt, s, s.block)) != SPARKATTN_OK) return rc;
  FwdParams prm;
  prm.kept_idx = kept_idx;
  prm.kept_cnt = kept_cnt;
  prm.q_scale = q_scale;
  prm.k_scale = k_scale;
  prm.v_scale = v_scale;
  prm.out = static_cast<__nv_bfloat16*>(out);
  prm.lse = lse;
  prm.status = static_cast<int32_t*>(workspace);
  prm.H = s.H;
  prm.N = s.N;
  prm.nb = (s.N + s.block - 1) / s.block;
  prm.kmax = kmax;
  prm.frame_tokens = frame_tokens;
  prm.window = window;
  prm.stride_b = s.stride_b;
  prm.stride_h = s.stride_h;
  prm.stride_n = s.stride_n;
  const float sc = s.softmax_scale > 0.0f ? s.softmax_scale : 1.0f / sqrtf((float)s.d);
  prm.scale_log2 = sc * 1.4426950408889634f;
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  return launch_fwd_t<64, 64, false>(s, mq, mk, mv, prm, stream);
}

}  // namespace sparkattn
