// sparkattn_fwd, d = 128 with 128-token blocks (bf16 and FP8): persistent block-sparse forward that works on
// TWO adjacent query blocks per CTA, one per softmax warpgroup.
//
// Arithmetic: Sec. 2 softmax attention restricted to the kept tiles (Sec. 4.1, sparse branch), fp32 online
// softmax, P rounded to the input precision for the second product: the same as fwd.cu.
//
// Schedule.  A work item is a pair of adjacent query blocks (2p, 2p+1) of one (batch, head).  Warpgroup g
// (warps 4-7 / 8-11, thread = query row) owns query block 2p+g for the whole item: its S accumulator, its
// running row maximum and row sum and its O accumulator are private, so nothing about a tile ever crosses
// from one warpgroup to the other.  TMEM: S_A | S_B | O_A | O_B (4 x 128 columns); P overlays S.
// A small pre-pass merges the two kept lists of a pair into one stream of K / V tile loads: a key block kept
// by both query blocks is loaded once and used by both ("shared"), the blocks kept by only one of them are
// interleaved A, B, A, B, ...; every warpgroup gets its own op list (key block, position in the load stream).
//   warp 0   TMA producer (one thread): Q_A, Q_B (one slot each), the K ring and the V ring in stream order.
//   warp 1   MMA issuer (one thread, polling): per warpgroup the strictly alternating sequence
//            S(0), PV(0), S(1), PV(1), ...; S_g(n+1) follows PV_g(n) in program order, which is what makes
//            P overlaying S safe (one thread's MMAs execute in order).  While warpgroup A computes the
//            softmax of its tile the tensor pipe runs PV and the next S of warpgroup B, and vice versa.
//   warps 2-3 idle.
// A ring slot is released by the MMA thread after its last consumer (the second one for a shared tile).
// Work items go to CTA c as c, c + grid, ... in head-major order (CTAs running together read one head's K/V
// from L2).  Every wait is bounded; nothing waits on another CTA.
#include <cuda.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "launch.h"
#include "tmap.h"

namespace sparkattn {

constexpr int kDuoThreads = 384;
constexpr int kDuoSoftmaxRegs = 216, kDuoCtrlRegs = 80;    // 2*128*216 + 128*80 = 384*168
constexpr int kDuoD = 128, kDuoBlk = 128;
constexpr float kDuoLazyLog2 = 8.0f;          // bf16: P may exceed 1 by up to 2^8 before O is rescaled
// FP8: P is pre-scaled by 2^4 * (s_v[j] / max s_v) and may grow by another 2^4 before O is rescaled:
// at most 2^8 = 256 < 448, the E4M3 maximum.
constexpr float kDuoFp8LazyLog2 = 4.0f, kDuoFp8PScaleLog2 = 4.0f;
constexpr int kDuoMaxBlocks = 16384;          // key blocks per head the list pre-pass can mark in shared memory
constexpr int kDuoListWarps = 4;

template <bool FP8>
struct DuoCfg {
  static constexpr int kTile = FP8 ? 16384 : 32768;            // bytes of one 128 x 128 input tile
  static constexpr int kRingK = FP8 ? 5 : 2, kRingV = FP8 ? 7 : 3;
  static constexpr int kOffQ = 0;                               // Q_A, Q_B
  static constexpr int kOffK = 2 * kTile;
  static constexpr int kOffV = kOffK + kRingK * kTile;
  static constexpr int kOffMisc = kOffV + kRingV * kTile;       // 224 KB in both precisions
  static constexpr int kSmem = kOffMisc + 64 * 8 /*barriers*/ + 64;
};

// op entry of a warpgroup's list: key block | position in the item's load stream << 16 | shared << 30
__device__ __forceinline__ int duo_op_kb(int e) { return e & 0xffff; }
__device__ __forceinline__ int duo_op_pos(int e) { return (e >> 16) & 0x1fff; }
__device__ __forceinline__ bool duo_op_shared(int e) { return ((e >> 30) & 1) != 0; }

struct DuoParams {
  const int4* hdr;             // [items] (ops of A, ops of B, tile loads, 0)
  const int32_t* ops;          // [items][2][kmax]
  const float* q_scale;        // FP8: [B*H*nb] dequantisation scales of the token blocks
  const float* k_scale;
  const float* v_scale;
  const float* v_max;          // FP8: [B*H] largest V scale of the head (pre-pass)
  __nv_bfloat16* out;
  float* lse;
  int32_t* status;
  int H, N, nb, items, nbq, kmax;
  int frame_tokens, window;    // causal frame window (0 = none)
  const int32_t* blk_valid;    // [nb] real tokens per block (bricks padded to whole blocks), or NULL
  int64_t stride_b, stride_h, stride_n;
  float scale_log2;
};

// ------------------------------------------------------------------ list pre-pass
// One warp per pair of query blocks.  Range-checks both kept lists (bad entries are reported and dropped,
// duplicates fold), splits their union into C = kept by both, OA = only by the first, OB = only by the
// second query block, and lays the load stream out as C then OA / OB interleaved (or the other way round
// when a query block's own key block is in its only-list): every query block meets its own key block as
// early as possible, which keeps the lazy rescale rare (a row's maximum is usually set there).
__global__ void __launch_bounds__(kDuoListWarps * 32)
duo_lists_kernel(const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ kept_cnt, int4* __restrict__ hdr,
                 int32_t* __restrict__ ops, int pairs, int nb, int nbq, int kmax, int32_t* status) {
  extern __shared__ uint32_t s_bits[];                      // [kDuoListWarps][2][words]
  const int words = (nb + 31) / 32;
  const int wl = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pair = blockIdx.x * kDuoListWarps + wl;
  if (pair >= pairs) return;
  uint32_t* bits = s_bits + wl * 2 * words;
  for (int i = lane; i < 2 * words; i += 32) bits[i] = 0u;
  __syncwarp();
  const int bh = pair / nbq, qp = pair % nbq;
  for (int side = 0; side < 2; ++side) {
    const int qb = 2 * qp + side;
    if (qb >= nb) break;
    const int64_t item = (int64_t)bh * nb + qb;
    const int cnt = kept_cnt ? min(max(__ldg(kept_cnt + item), 0), kmax) : kmax;
    const int32_t* src = kept_idx + item * kmax;
    for (int t = lane; t < cnt; t += 32) {
      const int kb = __ldg(src + t);
      if (kb >= 0 && kb < nb) atomicOr(bits + side * words + (kb >> 5), 1u << (kb & 31));
      else report_status(status, SPARKATTN_E_BAD_INDEX, kb);
    }
  }
  __syncwarp();
  const uint32_t* ba = bits;
  const uint32_t* bb = bits + words;
  int nC = 0, nOA = 0, nOB = 0;
  for (int wd = lane; wd < words; wd += 32) {
    const uint32_t a = ba[wd], b = bb[wd];
    nC += __popc(a & b); nOA += __popc(a & ~b); nOB += __popc(b & ~a);
  }
  nC = __reduce_add_sync(0xffffffffu, nC);
  nOA = __reduce_add_sync(0xffffffffu, nOA);
  nOB = __reduce_add_sync(0xffffffffu, nOB);
  const int own0 = 2 * qp, own1 = 2 * qp + 1;            // both in one bitmap word (own0 is even)
  auto has = [&](const uint32_t* bm, int kb) { return kb < nb && ((bm[kb >> 5] >> (kb & 31)) & 1u) != 0u; };
  const bool a0 = has(ba, own0), b0 = has(bb, own0), a1 = has(ba, own1), b1 = has(bb, own1);
  const bool only_first = (a0 && !b0) || (b1 && !a1);
  const int baseC = only_first ? nOA + nOB : 0, baseO = only_first ? 0 : nC;
  const int opC_a = only_first ? nOA : 0, opC_b = only_first ? nOB : 0, opO = only_first ? 0 : nC;
  int32_t* opa = ops + (int64_t)pair * 2 * kmax;
  int32_t* opb = opa + kmax;
  auto posOA = [&](int j) { return baseO + (j < nOB ? 2 * j : nOB + j); };
  auto posOB = [&](int j) { return baseO + (j < nOA ? 2 * j + 1 : nOA + j); };
  // own blocks first in their sublists
  int rC = 0, rOA = 0, rOB = 0;
  if (lane == 0) {
    if (a0 && b0) { opa[opC_a + rC] = opb[opC_b + rC] = own0 | ((baseC + rC) << 16) | (1 << 30); }
  }
  if (a0 && b0) ++rC;
  if (lane == 0) {
    if (a1 && b1) { opa[opC_a + rC] = opb[opC_b + rC] = own1 | ((baseC + rC) << 16) | (1 << 30); }
  }
  if (a1 && b1) ++rC;
  if (a0 && !b0) { if (lane == 0) opa[opO + rOA] = own0 | (posOA(rOA) << 16); ++rOA; }
  if (b1 && !a1) { if (lane == 0) opb[opO + rOB] = own1 | (posOB(rOB) << 16); ++rOB; }
  // the own blocks placed above leave the ascending scan
  const uint32_t ownmask_c = ((a0 && b0) ? 1u : 0u) | ((a1 && b1) ? 2u : 0u);
  const uint32_t ownmask_a = (a0 && !b0) ? 1u : 0u, ownmask_b = (b1 && !a1) ? 2u : 0u;
  const uint32_t lt = (1u << lane) - 1u;
  for (int base = 0; base < nb; base += 32) {
    const int kb = base + lane;
    const uint32_t a = ba[base >> 5], b = bb[base >> 5];
    uint32_t c = a & b, oa = a & ~b, ob = b & ~a;
    if (base == (own0 & ~31)) {
      c &= ~(ownmask_c << (own0 & 31));
      oa &= ~(ownmask_a << (own0 & 31));
      ob &= ~(ownmask_b << (own0 & 31));
    }
    if ((c >> lane) & 1u) {
      const int r = rC + __popc(c & lt);
      opa[opC_a + r] = opb[opC_b + r] = kb | ((baseC + r) << 16) | (1 << 30);
    }
    if ((oa >> lane) & 1u) {
      const int r = rOA + __popc(oa & lt);
      opa[opO + r] = kb | (posOA(r) << 16);
    }
    if ((ob >> lane) & 1u) {
      const int r = rOB + __popc(ob & lt);
      opb[opO + r] = kb | (posOB(r) << 16);
    }
    rC += __popc(c); rOA += __popc(oa); rOB += __popc(ob);
  }
  if (lane == 0) hdr[pair] = make_int4(nC + nOA, nC + nOB, nC + nOA + nOB, 0);
}

// FP8: largest V block scale of every (batch, head); one warp each
__global__ void duo_vmax_kernel(const float* __restrict__ v_scale, float* __restrict__ v_max, int bh_count, int nb) {
  const int bh = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (bh >= bh_count) return;
  float m = 0.0f;
  for (int j = lane; j < nb; j += 32) m = fmaxf(m, __ldg(v_scale + (int64_t)bh * nb + j));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) v_max[bh] = m;
}

// ------------------------------------------------------------------ device helpers
// Walks one warpgroup's op lists over the CTA's items, one entry ahead of its use; the next item's header and
// first entry are fetched while the current item runs.
struct DuoReader {
  const int4* hdr;
  const int32_t* ops;      // already offset by g * kmax
  int64_t lstride;         // 2 * kmax
  int g, item, step, items;
  int n, nloads, i, cur, nxt;
  int base;                // position of the item's first tile load in the CTA's load stream
  int ord;                 // items before this one in which this warpgroup had work
  int4 h_next;
  int first_next;

  __device__ __forceinline__ void prefetch_next() {
    const int nx = item + step;
    h_next = make_int4(0, 0, 0, 0);
    first_next = 0;
    if (nx < items) {
      h_next = __ldg(hdr + nx);
      first_next = __ldg(ops + (int64_t)nx * lstride);
    }
  }
  __device__ __forceinline__ void open() {
    i = 0;
    if (n > 1) nxt = __ldg(ops + (int64_t)item * lstride + 1);
    prefetch_next();
  }
  __device__ __forceinline__ void init(const DuoParams& p, int g_, int first_item, int step_) {
    hdr = p.hdr; ops = p.ops + (int64_t)g_ * p.kmax; lstride = 2 * (int64_t)p.kmax;
    g = g_; item = first_item; step = step_; items = p.items;
    base = 0; ord = 0; n = 0; nloads = 0; cur = 0; nxt = 0; i = 0;
    if (item < items) {
      const int4 h = __ldg(hdr + item);
      n = g ? h.y : h.x; nloads = h.z;
      cur = __ldg(ops + (int64_t)item * lstride);
      open();
    }
  }
  __device__ __forceinline__ bool done() const { return item >= items; }
  __device__ __forceinline__ bool item_end() const { return i >= n; }
  __device__ __forceinline__ void advance() {
    ++i;
    cur = nxt;
    if (i + 1 < n) nxt = __ldg(ops + (int64_t)item * lstride + i + 1);
  }
  __device__ __forceinline__ void next_item() {
    if (n > 0) ++ord;
    base += nloads;
    item += step;
    if (item < items) {
      n = g ? h_next.y : h_next.x; nloads = h_next.z;
      cur = first_next;
      open();
    }
  }
  __device__ __forceinline__ int pos() const { return base + duo_op_pos(cur); }
};

struct DuoIdle {
  uint64_t t0;
  uint32_t polls;
  __device__ __forceinline__ void reset() { polls = 0; }
  // Nothing was ready: yield the issue slots to the softmax warps of this scheduler for a moment.
  __device__ __forceinline__ bool idle(volatile int* abort_flag, int32_t* status, int wait_id) {
    if (polls == 0) t0 = global_timer_ns();
    __nanosleep(32);
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

// ------------------------------------------------------------------ the kernel
template <bool FP8, bool WINDOW>
__global__ void __launch_bounds__(kDuoThreads, 1)
fwd_duo_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const DuoParams p) {
  using Cfg = DuoCfg<FP8>;
  constexpr int kTile = Cfg::kTile, RK = Cfg::kRingK, RV = Cfg::kRingV;
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sQ = smem + Cfg::kOffQ;
  unsigned char* sK = smem + Cfg::kOffK;
  unsigned char* sV = smem + Cfg::kOffV;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffMisc);
  uint64_t* bar_q_full = bars + 0;      // [2] Q tile of warpgroup g has landed
  uint64_t* bar_q_free = bars + 2;      // [2] every S product of the item that reads it is complete
  uint64_t* bar_s_full = bars + 4;      // [2] S of warpgroup g's next tile is complete
  uint64_t* bar_p_full = bars + 6;      // [2] 128 arrivals: P written over S
  uint64_t* bar_pv_done = bars + 8;     // [2] PV of warpgroup g's last issued tile is complete
  uint64_t* bar_o_free = bars + 10;     // [2] 128 arrivals: warpgroup g has read its O accumulator
  uint64_t* bar_k_full = bars + 12;     // [RK]
  uint64_t* bar_k_free = bar_k_full + RK;
  uint64_t* bar_v_full = bar_k_free + RK;
  uint64_t* bar_v_free = bar_v_full + RV;
  static_assert(12 + 2 * (RK + RV) <= 64, "barrier area");
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 64);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_q_full + i, 1); mbar_init(bar_q_free + i, 1);
      mbar_init(bar_s_full + i, 1); mbar_init(bar_p_full + i, 128);
      mbar_init(bar_pv_done + i, 1); mbar_init(bar_o_free + i, 128);
    }
    for (int i = 0; i < RK; ++i) { mbar_init(bar_k_full + i, 1); mbar_init(bar_k_free + i, 1); }
    for (int i = 0; i < RV; ++i) { mbar_init(bar_v_full + i, 1); mbar_init(bar_v_free + i, 1); }
    int dead = (*reinterpret_cast<volatile int32_t*>(p.status) == SPARKATTN_E_DEVICE_TIMEOUT) ? 1 : 0;
    if ((smem_u32(smem) & 1023u) != 0u) {       // the swizzled tiles need a 1024-byte aligned base
      report_status(p.status, SPARKATTN_E_MISALIGNED, (int)(smem_u32(smem) & 1023u));
      dead = 1;
    }
    *s_abort = dead;
    mbar_fence_init();
  }
  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_k); tma_prefetch_desc(&tmap_v);
    }
    __syncwarp();
    tmem_alloc(s_tmem, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const bool dead = *s_abort != 0;
  const int first_item = blockIdx.x, item_step = gridDim.x;

  if (warp < 4) reg_dec<kDuoCtrlRegs>();
  if (dead) {
    // fall through to the teardown
  } else if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (one thread)
    if (lane == 0) {
      // Q cursor: per item, the Q tile of every warpgroup that has work in it
      int q_item = first_item, q_g = 0, q_ord[2] = {0, 0};
      int4 q_h = q_item < p.items ? __ldg(p.hdr + q_item) : make_int4(0, 0, 0, 0);
      int4 q_hn = q_item + item_step < p.items ? __ldg(p.hdr + q_item + item_step) : make_int4(0, 0, 0, 0);
      // K and V cursors over the merged load stream of both warpgroups
      struct Stream {
        DuoReader a, b;
        int rel, slot, phase, count;       // next load of the item; its ring slot and the slot's use count parity
      };
      Stream ks, vs;
      ks.a.init(p, 0, first_item, item_step); ks.b.init(p, 1, first_item, item_step);
      vs.a.init(p, 0, first_item, item_step); vs.b.init(p, 1, first_item, item_step);
      ks.rel = vs.rel = 0; ks.slot = vs.slot = 0; ks.phase = vs.phase = 0; ks.count = vs.count = 0;
      auto next_kb = [&](Stream& s) {
        const bool from_a = !s.a.item_end() && duo_op_pos(s.a.cur) == s.rel;
        const bool from_b = !s.b.item_end() && duo_op_pos(s.b.cur) == s.rel;
        const int kb = from_a ? duo_op_kb(s.a.cur) : duo_op_kb(s.b.cur);
        if (from_a) s.a.advance();
        if (from_b) s.b.advance();
        ++s.rel;
        return kb;
      };
      auto load_tile = [&](unsigned char* dst, const CUtensorMap* map, uint64_t* bar, int row0, int item) {
        const int bh = item / p.nbq;
        const int hh = bh % p.H, bb = bh / p.H;
        mbar_expect_tx(bar, kTile);
        tma_load_4d(dst, map, bar, 0, row0, hh, bb);
        if constexpr (!FP8) tma_load_4d(dst + kTile / 2, map, bar, 64, row0, hh, bb);
      };
      bool ok = true;
      DuoIdle guard;
      guard.reset();
      while (ok && (q_item < p.items || !ks.a.done() || !vs.a.done())) {
        bool progressed = false;
        // all barrier tests first, back to back (a test is a shared-memory round trip)
        const bool qf = q_ord[q_g] == 0 ? true : mbar_test(bar_q_free + q_g, (q_ord[q_g] - 1) & 1);
        const bool kf = ks.count < RK ? true : mbar_test(bar_k_free + ks.slot, ks.phase ^ 1);
        const bool vf = vs.count < RV ? true : mbar_test(bar_v_free + vs.slot, vs.phase ^ 1);
        if (q_item < p.items) {
          const int ng = q_g ? q_h.y : q_h.x;
          if (ng == 0) {
            if (++q_g == 2) {
              q_g = 0; q_item += item_step; q_h = q_hn;
              q_hn = q_item + item_step < p.items ? __ldg(p.hdr + q_item + item_step) : make_int4(0, 0, 0, 0);
            }
            progressed = true;
          } else if (qf) {
            const int qb = 2 * (q_item % p.nbq) + q_g;
            load_tile(sQ + q_g * kTile, &tmap_q, bar_q_full + q_g, qb * kDuoBlk, q_item);
            ++q_ord[q_g];
            if (++q_g == 2) {
              q_g = 0; q_item += item_step; q_h = q_hn;
              q_hn = q_item + item_step < p.items ? __ldg(p.hdr + q_item + item_step) : make_int4(0, 0, 0, 0);
            }
            progressed = true;
          }
        }
        if (!ks.a.done()) {
          if (ks.rel >= ks.a.nloads) {
            ks.a.next_item(); ks.b.next_item(); ks.rel = 0;
            progressed = true;
          } else if (kf) {
            const int item = ks.a.item;
            const int kb = next_kb(ks);
            load_tile(sK + ks.slot * kTile, &tmap_k, bar_k_full + ks.slot, kb * kDuoBlk, item);
            ++ks.count;
            if (++ks.slot == RK) { ks.slot = 0; ks.phase ^= 1; }
            progressed = true;
          }
        }
        if (!vs.a.done()) {
          if (vs.rel >= vs.a.nloads) {
            vs.a.next_item(); vs.b.next_item(); vs.rel = 0;
            progressed = true;
          } else if (vf) {
            const int item = vs.a.item;
            const int kb = next_kb(vs);
            load_tile(sV + vs.slot * kTile, &tmap_v, bar_v_full + vs.slot, kb * kDuoBlk, item);
            ++vs.count;
            if (++vs.slot == RV) { vs.slot = 0; vs.phase ^= 1; }
            progressed = true;
          }
        }
        if (progressed) guard.reset();
        else ok = guard.idle(s_abort, p.status, 1);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (one thread)
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(FP8 ? 0u : 1u, 128, kDuoBlk, false);
      constexpr uint32_t idesc_pv = make_idesc(FP8 ? 0u : 1u, 128, kDuoD, true);
      constexpr int kPvSteps = FP8 ? 4 : 8;          // 32 bytes of P per row per MMA: 16 bf16 or 32 E4M3 keys
      DuoReader rd[2];
      rd[0].init(p, 0, first_item, item_step);
      rd[1].init(p, 1, first_item, item_step);
      bool pv_next[2] = {false, false};              // the warpgroup's next op: S (false) or PV (true) of op rd[g].i
      int tcount[2] = {0, 0};                        // tiles of the warpgroup issued so far (barrier phases)
      uint32_t k_once = 0u, v_once = 0u;             // ring slots whose shared tile has had its first consumer
      bool ok = true;
      DuoIdle guard;
      guard.reset();
      while (ok && (!rd[0].done() || !rd[1].done())) {
        bool progressed = false;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          DuoReader& r = rd[g];
          if (r.done()) continue;
          if (!pv_next[g] && r.item_end()) {
            r.next_item();
            progressed = true;
            continue;
          }
          const int pos = r.pos();
          if (pv_next[g]) {
            const int vslot = pos % RV;
            const bool pf = mbar_test(bar_p_full + g, tcount[g] & 1);
            const bool vf = mbar_test(bar_v_full + vslot, (pos / RV) & 1);
            // first tile of an item: the warpgroup must have read the previous item's O
            const bool of = (r.i > 0 || r.ord == 0) ? true : mbar_test(bar_o_free + g, (r.ord - 1) & 1);
            if (pf && vf && of) {
              tc_fence_after();
              const uint64_t dV = make_smem_desc_sw128(smem_u32(sV + vslot * kTile), kTile / 2);
              const uint32_t v_lo = (uint32_t)dV, v_hi = (uint32_t)(dV >> 32);
              const uint32_t tO = tmem + 256 + g * 128, tP = tmem + g * 128;
#pragma unroll
              for (int kk = 0; kk < kPvSteps; ++kk)
                mma_ts<FP8>(tO, tP + kk * 8, make_desc(v_lo + ((kk * (128 / kPvSteps) * 128) >> 4), v_hi), idesc_pv,
                            (r.i == 0 && kk == 0) ? 0u : 1u);
              tc_commit(bar_pv_done + g);
              bool release = true;
              if (duo_op_shared(r.cur)) {
                release = ((v_once >> vslot) & 1u) != 0u;
                v_once ^= 1u << vslot;
              }
              if (release) tc_commit(bar_v_free + vslot);
              ++tcount[g];
              r.advance();
              pv_next[g] = false;
              progressed = true;
            }
          }
          if (!pv_next[g] && !r.item_end()) {
            const int kpos = r.pos();
            const int kslot = kpos % RK;
            const bool kf = mbar_test(bar_k_full + kslot, (kpos / RK) & 1);
            const bool qf = r.i > 0 ? true : mbar_test(bar_q_full + g, r.ord & 1);
            if (kf && qf) {
              tc_fence_after();
              const uint64_t dQ = make_smem_desc_sw128(smem_u32(sQ + g * kTile), 16);
              const uint64_t dK = make_smem_desc_sw128(smem_u32(sK + kslot * kTile), 16);
              const uint32_t q_lo = (uint32_t)dQ, q_hi = (uint32_t)(dQ >> 32), k_lo = (uint32_t)dK, k_hi = (uint32_t)(dK >> 32);
              // 32 bytes of the channel dimension per MMA: 16 bf16 (8 MMAs over two slabs) or 32 E4M3 (4 MMAs)
#pragma unroll
              for (int sl = 0; sl < (FP8 ? 1 : 2); ++sl)
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                  mma_ss<FP8>(tmem + g * 128, make_desc(q_lo + ((sl * (kTile / 2) + kk * 32) >> 4), q_hi),
                              make_desc(k_lo + ((sl * (kTile / 2) + kk * 32) >> 4), k_hi), idesc_qk, (sl | kk) != 0 ? 1u : 0u);
              tc_commit(bar_s_full + g);
              bool release = true;
              if (duo_op_shared(r.cur)) {
                release = ((k_once >> kslot) & 1u) != 0u;
                k_once ^= 1u << kslot;
              }
              if (release) tc_commit(bar_k_free + kslot);
              if (r.i == r.n - 1) tc_commit(bar_q_free + g);     // the item's last S of this warpgroup: its Q slot can be refilled
              pv_next[g] = true;
              progressed = true;
            }
          }
        }
        if (progressed) guard.reset();
        else ok = guard.idle(s_abort, p.status, 2);
      }
    }
  } else if (warp >= 4) {
    // ----------------------------------------------------------------- softmax warpgroups
    reg_inc<kDuoSoftmaxRegs>();
    const int g = (warp >> 2) - 1;                    // warpgroup = query block of the pair
    const int row = threadIdx.x & 127;                // query row inside the block = TMEM lane
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + g * 128 + lane_off, tO = tmem + 256 + g * 128 + lane_off;
    constexpr float kLazy = FP8 ? kDuoFp8LazyLog2 : kDuoLazyLog2;
    DuoReader r;
    r.init(p, g, first_item, item_step);
    int tcount = 0;                                   // tiles of this warpgroup done so far (barrier phases)
    bool ok = true;
    for (; ok && !r.done(); r.next_item()) {
      const int item = r.item, n = r.n;
      const int qp = item % p.nbq, bh = item / p.nbq;
      const int qb = 2 * qp + g;
      if (qb >= p.nb) continue;                       // the odd last pair has no second query block
      const int h = bh % p.H, b = bh / p.H;
      const int q_row = qb * kDuoBlk + row;
      const bool row_valid = q_row < p.N;
      __nv_bfloat16* orow = p.out + b * p.stride_b + h * p.stride_h + (int64_t)q_row * p.stride_n;
      if (n == 0) {
        // empty kept list: zero output, lse = -inf
        if (row_valid) {
#pragma unroll
          for (int ch = 0; ch < kDuoD / 8; ++ch) reinterpret_cast<uint4*>(orow)[ch] = make_uint4(0u, 0u, 0u, 0u);
          if (p.lse) p.lse[(int64_t)bh * p.N + q_row] = -INFINITY;
        }
        continue;
      }
      // keys this row may attend to: [klo, khi) (everything up to N without a causal window)
      int klo = 0, khi = p.N;
      if constexpr (WINDOW) {
        const int fi = min(q_row, p.N - 1) / p.frame_tokens;
        klo = max(fi - p.window + 1, 0) * p.frame_tokens;
        khi = (int)min((long long)(fi + 1) * p.frame_tokens, (long long)p.N);
      }
      float m_used = -INFINITY, l = 0.0f;             // running reference maximum (log2 units) and row sum relative to it
      float q_sc = 1.0f, v_max = 1.0f;
      const float* ksc = FP8 ? p.k_scale + (int64_t)bh * p.nb : nullptr;
      const float* vsc = FP8 ? p.v_scale + (int64_t)bh * p.nb : nullptr;
      float ks_nx = 1.0f, vs_nx = 1.0f;               // scales of the tile after this one are fetched a tile ahead
      int bv_nx = kDuoBlk;
      if constexpr (FP8) {
        q_sc = __ldg(p.q_scale + (int64_t)bh * p.nb + qb);
        v_max = __ldg(p.v_max + bh);
        ks_nx = __ldg(ksc + duo_op_kb(r.cur));
        vs_nx = __ldg(vsc + duo_op_kb(r.cur));
      }
      if (p.blk_valid != nullptr) bv_nx = __ldg(p.blk_valid + duo_op_kb(r.cur));
      const float inv_vmax = 1.0f / v_max;
      for (; ok && !r.item_end(); r.advance(), ++tcount) {
        const int kb = duo_op_kb(r.cur);
        const float ks0 = ks_nx, vs0 = vs_nx;
        const int bv0 = bv_nx;
        if (r.i + 1 < n) {
          const int kbn = duo_op_kb(r.nxt);
          if constexpr (FP8) { ks_nx = __ldg(ksc + kbn); vs_nx = __ldg(vsc + kbn); }
          if (p.blk_valid != nullptr) bv_nx = __ldg(p.blk_valid + kbn);
        }
        float c = p.scale_log2;                      // logit -> log2 units
        float p_off = 0.0f;                          // log2 of the factor folded into P
        if constexpr (FP8) {
          c *= q_sc * ks0;
          p_off = kDuoFp8PScaleLog2 + log2f(vs0 * inv_vmax);
        }
        // this row's valid columns of the tile: [c_lo, c_hi)
        const int c_lo = klo - kb * kDuoBlk, c_hi = min(khi - kb * kDuoBlk, bv0);
        ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full + g, tcount & 1, s_abort, p.status, 4));
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[kDuoBlk];
#pragma unroll
        for (int ch = 0; ch < kDuoBlk / 32; ++ch) tmem_ld32(tS + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[ch * 32]));
        tc_wait_ld();
        if ((WINDOW && c_lo > 0) || c_hi < kDuoBlk) {   // ragged last key block / padding rows of a brick / keys outside the causal window get weight 0
          if (!WINDOW && c_hi >= kDuoBlk - 32) {        // a short tail (every tile of a padded brick layout): 32 tests, not 128
#pragma unroll
            for (int i = kDuoBlk - 32; i < kDuoBlk; ++i)
              if (i >= c_hi) sr[i] = 0xff800000u;
          } else {
#pragma unroll
            for (int i = 0; i < kDuoBlk; ++i)
              if ((WINDOW && i < c_lo) || i >= c_hi) sr[i] = 0xff800000u;
          }
        }
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]);
        float mx2 = __uint_as_float(sr[2]), mx3 = __uint_as_float(sr[3]);
#pragma unroll
        for (int i = 4; i < kDuoBlk; i += 8) {
          mx0 = fmax3(mx0, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
          mx1 = fmax3(mx1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
          if (i + 4 < kDuoBlk) {
            mx2 = fmax3(mx2, __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
            mx3 = fmax3(mx3, __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
          }
        }
        const float m_tile = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * c;
        bool need = false;
        float alpha = 1.0f;
        if (m_used == -INFINITY) {
          m_used = m_tile;                 // nothing accumulated for this row yet: O row and l are 0
        } else if (m_tile > m_used + kLazy) {
          alpha = fast_exp2(m_used - m_tile);
          l *= alpha;
          m_used = m_tile;
          need = true;
        }
        if (__any_sync(0xffffffffu, need)) {
          // O is rescaled only when no PV of this warpgroup is in flight: the last one issued is the previous
          // tile's (this tile's follows the P written below)
          ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + g, (tcount - 1) & 1, s_abort, p.status, 6));
          if (!ok) break;
          tc_fence_after();
          const uint64_t a2 = pack_f32x2(alpha, alpha);
#pragma unroll 1
          for (int ch = 0; ch < kDuoD / 32; ++ch) {
            uint32_t rr[32];
            tmem_ld32(tO + ch * 32, rr);
            tc_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float2 o2 = unpack_f32x2(fmul2(pack_f32x2(__uint_as_float(rr[i]), __uint_as_float(rr[i + 1])), a2));
              rr[i] = __float_as_uint(o2.x);
              rr[i + 1] = __float_as_uint(o2.y);
            }
            tmem_st32(tO + ch * 32, rr);
          }
          tc_wait_st();
        }

        // P = exp2(S*c - m) in the input precision over the start of the S columns (S is in registers; every
        // earlier PV of this warpgroup is complete, because this tile's S ran after it on the same pipe)
        const float neg_m = m_used == -INFINITY ? 0.0f : p_off - m_used;     // a fully masked row: exp2(-inf) = 0, not NaN
        const uint64_t c2 = pack_f32x2(c, c), nm2 = pack_f32x2(neg_m, neg_m);
        uint64_t lsum0 = pack_f32x2(0.0f, 0.0f), lsum1 = lsum0;
        constexpr int kWords = FP8 ? 8 : 16;        // 32-bit words of P per 32 S columns
#pragma unroll
        for (int ch = 0; ch < kDuoBlk / 32; ++ch) {
          uint32_t w[kWords];
          float e[32];
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float2 x = unpack_f32x2(
                ffma2(pack_f32x2(__uint_as_float(sr[ch * 32 + i]), __uint_as_float(sr[ch * 32 + i + 1])), c2, nm2));
            e[i] = fast_exp2(x.x);
            e[i + 1] = fast_exp2(x.y);
            if (((i >> 1) & 1) != 0) lsum1 = fadd2(lsum1, pack_f32x2(e[i], e[i + 1]));
            else lsum0 = fadd2(lsum0, pack_f32x2(e[i], e[i + 1]));
          }
          if constexpr (FP8) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(e[4 * i], e[4 * i + 1]), __NV_SATFINITE, __NV_E4M3);
              const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(e[4 * i + 2], e[4 * i + 3]), __NV_SATFINITE, __NV_E4M3);
              w[i] = lo | (hi << 16);
            }
            tmem_st8(tS + ch * 8, w);
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(e[2 * i], e[2 * i + 1]);
              w[i] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            tmem_st16(tS + ch * 16, w);
          }
        }
        {
          const float2 ls = unpack_f32x2(fadd2(lsum0, lsum1));
          if constexpr (FP8) l += (ls.x + ls.y) * fast_exp2(-p_off);      // the row sum is kept without the factor folded into P
          else l += ls.x + ls.y;
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_full + g);
      }
      if (!ok) break;

      // ------------------------------------------------------------ end of the item: O / l -> global memory
      ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + g, (tcount - 1) & 1, s_abort, p.status, 9));
      if (!ok) break;
      tc_fence_after();
      float inv = l > 0.0f ? 1.0f / l : 0.0f;           // no admissible key at all: zero row, lse = -inf
      if constexpr (FP8) inv *= v_max * 0.0625f;        // undo the 2^4 / max s_v folded into P
#pragma unroll 1
      for (int ch = 0; ch < kDuoD / 32; ++ch) {
        uint32_t rr[32];
        tmem_ld32(tO + ch * 32, rr);
        tc_wait_ld();
        if (ch == kDuoD / 32 - 1) {
          tc_fence_before();
          mbar_arrive(bar_o_free + g);                  // the accumulator is in registers: the next item's first PV may overwrite it
        }
        if (row_valid) {
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            uint32_t ww[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(rr[8 * cc + 2 * j]) * inv,
                                                              __uint_as_float(rr[8 * cc + 2 * j + 1]) * inv);
              ww[j] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            reinterpret_cast<uint4*>(orow + ch * 32)[cc] = make_uint4(ww[0], ww[1], ww[2], ww[3]);
          }
        }
      }
      if (row_valid && p.lse) p.lse[(int64_t)bh * p.N + q_row] = (m_used + log2f(l)) * 0.6931471805599453f;
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    if (*s_abort) __nanosleep(200000);  // let copies / MMAs in flight land before the CTA's resources go
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ------------------------------------------------------------------ host side
bool fwd_duo_supported(const sparkattn_shape_t& s) {
  return s.d == 128 && s.block == 128 && (s.N + 127) / 128 <= kDuoMaxBlocks;
}

size_t fwd_duo_workspace_bytes(const sparkattn_shape_t& s, int kmax) {
  const int nb = (s.N + s.block - 1) / s.block;
  const size_t items = (size_t)s.B * s.H * ((nb + 1) / 2);
  // header | (ops A, ops B, loads) per pair | the two op lists of every pair | FP8: largest V scale per (batch, head)
  return kWorkspaceHeaderBytes + (items * 16 + 255) / 256 * 256 + (items * 2 * (size_t)kmax * 4 + 255) / 256 * 256 +
         (size_t)s.B * s.H * 4;
}

int launch_fwd_duo(const sparkattn_shape_t& s, bool fp8, const void* q, const void* k, const void* v,
                   const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                   const int32_t* kept_cnt, int kmax, int frame_tokens, int window, const int32_t* block_valid,
                   void* out, float* lse, void* workspace, cudaStream_t stream) {
  CUtensorMap mq, mk, mv;
  int rc;
  const int elt = fp8 ? 1 : 2;
  if ((rc = make_token_map(&mq, q, elt, s, kDuoBlk)) != SPARKATTN_OK) return rc;
  if ((rc = make_token_map(&mk, k, elt, s, kDuoBlk)) != SPARKATTN_OK) return rc;
  if ((rc = make_token_map(&mv, v, elt, s, kDuoBlk)) != SPARKATTN_OK) return rc;
  const int nb = (s.N + s.block - 1) / s.block;
  const int nbq = (nb + 1) / 2;
  const long long items = (long long)s.B * s.H * nbq;
  if (items > 0x7fffffffLL || kmax > 4096) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  char* base = static_cast<char*>(workspace);
  const size_t off_ops = kWorkspaceHeaderBytes + ((size_t)items * 16 + 255) / 256 * 256;
  const size_t off_vmax = off_ops + ((size_t)items * 2 * kmax * 4 + 255) / 256 * 256;
  DuoParams prm;
  prm.hdr = reinterpret_cast<const int4*>(base + kWorkspaceHeaderBytes);
  prm.ops = reinterpret_cast<const int32_t*>(base + off_ops);
  prm.q_scale = q_scale; prm.k_scale = k_scale; prm.v_scale = v_scale;
  prm.v_max = reinterpret_cast<const float*>(base + off_vmax);
  prm.out = static_cast<__nv_bfloat16*>(out);
  prm.lse = lse;
  prm.status = static_cast<int32_t*>(workspace);
  prm.H = s.H; prm.N = s.N; prm.nb = nb; prm.items = (int)items; prm.nbq = nbq; prm.kmax = kmax;
  prm.frame_tokens = frame_tokens; prm.window = window;
  prm.blk_valid = block_valid;
  prm.stride_b = s.stride_b; prm.stride_h = s.stride_h; prm.stride_n = s.stride_n;
  const float sc = s.softmax_scale > 0.0f ? s.softmax_scale : 1.0f / sqrtf((float)s.d);
  prm.scale_log2 = sc * 1.4426950408889634f;
  const int sm_count = current_sm_count();
  if (sm_count < 1) return SPARKATTN_E_CUDA;
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  const size_t bits = (size_t)kDuoListWarps * 2 * ((nb + 31) / 32) * sizeof(uint32_t);
  duo_lists_kernel<<<(unsigned)((items + kDuoListWarps - 1) / kDuoListWarps), kDuoListWarps * 32, bits, stream>>>(
      kept_idx, kept_cnt, reinterpret_cast<int4*>(base + kWorkspaceHeaderBytes), reinterpret_cast<int32_t*>(base + off_ops),
      (int)items, nb, nbq, kmax, prm.status);
  if (fp8)
    duo_vmax_kernel<<<(unsigned)((s.B * s.H + 7) / 8), 256, 0, stream>>>(v_scale, reinterpret_cast<float*>(base + off_vmax),
                                                                        s.B * s.H, nb);
  const bool win = frame_tokens > 0;
  auto kern = fp8 ? (win ? fwd_duo_kernel<true, true> : fwd_duo_kernel<true, false>)
                  : (win ? fwd_duo_kernel<false, true> : fwd_duo_kernel<false, false>);
  const int smem = fp8 ? DuoCfg<true>::kSmem : DuoCfg<false>::kSmem;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return SPARKATTN_E_CUDA;
  const unsigned grid = (unsigned)(items < sm_count ? items : sm_count);
  kern<<<grid, kDuoThreads, smem, stream>>>(mq, mk, mv, prm);
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

}  // namespace sparkattn
