// sparkattn_fwd, d = 128 (128-token blocks, or 64-token blocks in pairs; bf16 and FP8): persistent pipelined
// block-sparse forward.
//
// Same arithmetic as fwd.cu (Sec. 2 softmax attention restricted to the kept tiles, Sec. 4.1 sparse
// branch); different schedule.  Measured on the one-item-per-CTA kernel: a tile's chain
// S-MMA -> softmax -> PV-MMA is ~3300 clocks long even with the SM to itself, so two independent
// chains per SM leave the tensor pipe ~45 % busy.  Here one CTA per SM keeps the chain open: each
// softmax warpgroup owns an S buffer and a separate P buffer in TMEM (S0 | S1 | P0 | P1 | O =
// 128 + 128 + 64 + 64 + 128 columns), so its S buffer is free again as soon as the S row sits in
// registers and the next-but-one S product runs while the warpgroup is still busy with this tile:
//   warps 4-7 / 8-11 two softmax warpgroups; the tiles of the CTA's item stream alternate between
//                    them (global tile counter parity), thread r owns query row r.  The running
//                    reference maximum of a row travels from the warpgroup of tile t-1 to the
//                    warpgroup of tile t through shared memory (token barrier); it only moves
//                    when a tile maximum exceeds it by more than 2^8 (lazy rescale), and the
//                    warpgroup that moves it rescales O before it passes the token on.  Each
//                    warpgroup keeps its own partial row sum relative to the last reference it
//                    saw; the warpgroup of the item's last tile combines them, normalises O into
//                    the item's (now dead) Q slot and stores it with one TMA copy.
//   warp 0           TMA producer (one thread): Q (2 slots) and the K ring (2 slots; FP8: 4).
//   warp 3           TMA producer (one thread): the V ring (3 slots; FP8: 6).  Each producer sleeps in
//                    the wait for the slot it fills next (one thread polling all rings with a
//                    back-off answered a freed slot up to a microsecond late).
//   warp 1           S issuer: S = Q K^T of the next tile once its K has landed and its S buffer is
//                    free (the warpgroup holds the row of the tile two back in registers).
//   warp 2           PV issuer: O += P V of the oldest tile once its P is written.
//                    Two issuing warps on two schedulers: an issuing thread shares its scheduler
//                    with two softmax warps that are almost always ready and only gets an issue
//                    slot when they stall, so its instruction count per tile is what matters.
//                    Both sleep in their barrier waits (everything a product needs is needed).
// Work items (batch, head, query block) go to CTA c as c, c + grid, ... in head-major order, so
// the CTAs running together read K/V of one head from L2.  Kept lists are range-checked and
// compacted by a small pre-pass into the workspace; every role reads the clean lists from there.
// Every wait is bounded; nothing here waits on another CTA.
//
// EPI variant (kept lists of at most kEpiMaxKept blocks): 512 threads, warps 12-15 are a closing
// warpgroup.  At the end of an item the softmax warpgroups only leave their partial row sums (the
// warpgroup of the last tile in the first KB of the item's dead Q slot, the other one in s_lsum) and go
// on to the next item's tiles; the closing warpgroup waits for the last PV, reads O, normalises it into
// the Q slot, hands O back to the PV issuer, writes lse and stores the tile.  That takes the wait for the
// last PV, the O read and the store off the warpgroup whose next tile the pipeline needs (bf16 -2.6 %,
// FP8 -1 % at 18 tiles per item, 6-8 % at 6); with four more warps resident, and 40 registers for the
// control warps, the tile loop itself runs 3 % slower, so the launcher keeps the 384-thread kernel for
// longer lists.
//
// GATE variant (sparkattn_fwd_gated; bf16, 128-token blocks, 384 threads): the closing softmax warpgroup
// adds the gated low-rank term of Sec. 4.1 before the store.  Once the last PV of the item is complete it
// issues T = Q P_q^T (Q still in its slot) into its own P buffer, turns T into q~ = R(p) silu(T) as bf16 in
// place (rotary factors requested before the wait for T), reads O, issues y = q~ C (q~ from TMEM, C as
// bf16 in shared memory) over the O columns, and writes O_s + g r y / rms(y) into the Q slot.  P_q
// (16 KB) and C (16 KB) of the current (batch, head) take the place of the third V slot.  Arithmetic
// and order are those of comp.cu's apply pass, so the result equals the two separate calls bit for
// bit.  Measured (720p shape, 97 % sparsity): the closing grows from ~1300 to ~7200 clocks per item
// (two dependent tensor-core round trips, 128 special-function operations per row, three passes over
// TMEM), during which the pipeline drains: the fused call takes as long as the two calls it replaces.
#include <cuda.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "launch.h"
#include "rope.cuh"
#include "tmap.h"

namespace sparkattn {

constexpr int kPipeThreads = 384;                           // GATE variant: 4 control warps + 2 softmax warpgroups
constexpr int kPipeSoftmaxRegs = 216, kPipeCtrlRegs = 64;   // 2*128*216 + 128*64 <= 384*168
// short kept lists (EPI): a third warpgroup (warps 12-15) closes the items, see below
constexpr int kEpiThreads = 512;
constexpr int kEpiMaxKept = 32;                             // longest kept list the launcher gives to that variant
constexpr int kEpiSoftmaxRegs = 216, kEpiCtrlRegs = 40, kEpiCloseRegs = 40;   // 2*128*216 + 128*40 + 128*40 = 512*128
constexpr int kPD = 128, kPBLK = 128;
constexpr float kPipeLazyLog2 = 8.0f;        // bf16: P may exceed 1 by up to 2^8 before O is rescaled
// FP8: P is pre-scaled by 2^4 * (s_v[j] / max s_v) and may grow by another 2^4 before O is rescaled:
// at most 2^8 = 256 < 448, the E4M3 maximum; values below 2^-13 of the row maximum flush to zero.
constexpr float kPipeFp8LazyLog2 = 4.0f, kPipeFp8PScaleLog2 = 4.0f;
constexpr int kTile = 32768;                               // bytes of one 128 x 128 bf16 tile (two 64-column slabs)
constexpr int kOffQ = 0, kOffK = 2 * kTile, kOffMisc = 7 * kTile;     // Q slots | K ring, V ring (5 x 32 KB) | barriers ...
constexpr int kPipeSmem = kOffMisc + 512 /*barriers*/ + 2 * 128 * 4 /*reference maxima*/ + 128 * 8 /*row sums*/ + 64;

struct PipeParams {
  const int32_t* clean_cnt;    // [items] valid kept blocks per item
  const int32_t* clean_list;   // [items][kmax] their indices, compacted in list order
  const float* q_scale;        // FP8: [B*H*nb] dequantisation scales of the token blocks
  const float* k_scale;
  const float* v_scale;
  const float* v_max;          // FP8: [B*H] largest V scale of the head (pre-pass)
  __nv_bfloat16* out;
  float* lse;
  int32_t* status;
  int H, N, nb, items;
  int nbq;                     // work items per (batch, head): query blocks, or pairs of 64-token query blocks
  int lstride;                 // list entries per item in clean_list
  int frame_tokens, window;    // causal frame window (0 = none): key frame in (query frame - window, query frame]
  const int32_t* blk_valid;    // [nb] real tokens per block (bricks padded to whole blocks), or NULL
  int64_t stride_b, stride_h, stride_n;
  float scale_log2;
  // fused gate epilogue (GATE instantiation only; Sec. 4.1: O = O_s + g * r * RMSNorm(q~ C))
  RopeTable rope;
  const float2* rope_table;    // [T + Hg + Wg][rank/2] (cos, sin)
  const float* state;          // [B*H][rank][d] fp32
  const float* gate;           // [B*H][N]
  float eps;
};

// one warp per item: drop (and report) kept indices outside [0, nb), clamp the count, own block first
__global__ void compact_lists_kernel(const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ kept_cnt,
                                     int32_t* __restrict__ clean_cnt, int32_t* __restrict__ clean_list, int items,
                                     int nb, int kmax, int32_t* status) {
  const int item = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (item >= items) return;
  const int cnt = kept_cnt ? min(max(__ldg(kept_cnt + item), 0), kmax) : kmax;
  const int32_t* src = kept_idx + (int64_t)item * kmax;
  int32_t* dst = clean_list + (int64_t)item * kmax;
  int out = 0;
  for (int base = 0; base < cnt; base += 32) {
    const int t = base + lane;
    const int kb = (t < cnt) ? __ldg(src + t) : 0;
    const bool valid = (t < cnt) && kb >= 0 && kb < nb;
    if (t < cnt && !valid) report_status(status, SPARKATTN_E_BAD_INDEX, kb);
    const uint32_t ballot = __ballot_sync(0xffffffffu, valid);
    if (valid) dst[out + __popc(ballot & ((1u << lane) - 1u))] = kb;
    out += __popc(ballot);
  }
  if (lane == 0) clean_cnt[item] = out;
  // The query block's own key block goes first.  The result does not depend on the order of the tiles, the
  // work does: a row's running maximum is usually set by its own block, and when that block comes late (it is
  // the last entry of an ascending list under a causal window) nearly every row's maximum jumps past the lazy
  // threshold there and the whole O tile is rescaled; with it first the later tiles stay below the reference.
  __syncwarp();
  const int qb = item % nb;
  int p = -1;
  for (int base = 0; base < out && p < 0; base += 32) {
    const int t = base + lane;
    const uint32_t hit = __ballot_sync(0xffffffffu, t < out && dst[t] == qb);
    if (hit) p = base + __ffs(hit) - 1;
  }
  if (p > 0) {
    for (int base = (p / 32) * 32; base >= 0; base -= 32) {      // shift entries 0..p-1 up by one, highest chunk first
      const int t = base + lane;
      const bool mine = t <= p;
      int val = 0;
      if (mine) val = (t == 0) ? qb : dst[t - 1];
      __syncwarp();
      if (mine) dst[t] = val;
      __syncwarp();
    }
  }
}

// 64-token blocks: the kernel works on pairs of adjacent query blocks (128 query rows, the MMA's M) and on
// tiles of two key blocks.  One warp per pair merges the two kept lists (range-checked, duplicates folded)
// into one ascending list; an entry is block | in-list-of-first-query-block << 30 | in-list-of-second << 31,
// two entries per tile (an odd tail repeats its block with both flags clear).  clean_cnt = tiles.
constexpr int kPairMaxBlocks = 16384;    // key blocks per head the merge can mark in shared memory
constexpr int kPairWarps = 4;
__global__ void __launch_bounds__(kPairWarps * 32)
pair_lists_kernel(const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ kept_cnt,
                  int32_t* __restrict__ clean_cnt, int32_t* __restrict__ clean_list, int pairs, int nb, int nbq,
                  int kmax, int32_t* status) {
  extern __shared__ uint32_t s_bits[];                      // [kPairWarps][2][words]
  const int words = (nb + 31) / 32;
  const int wl = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pair = blockIdx.x * kPairWarps + wl;
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
  int32_t* dst = clean_list + (int64_t)pair * (2 * kmax);
  int out = 0;
  // the pair's own two key blocks first (see compact_lists_kernel), then the rest in ascending order
  const int own0 = 2 * qp;
  for (int kb = own0; kb <= own0 + 1 && kb < nb; ++kb) {
    const bool ina = (bits[kb >> 5] >> (kb & 31)) & 1u, inb = (bits[words + (kb >> 5)] >> (kb & 31)) & 1u;
    if (ina || inb) {
      if (lane == 0) dst[out] = kb | (ina ? (1 << 30) : 0) | (inb ? (int)(1u << 31) : 0);
      ++out;
    }
  }
  for (int base = 0; base < nb; base += 32) {
    const int kb = base + lane;
    const uint32_t a = bits[base >> 5], bmask = bits[words + (base >> 5)];
    const bool ina = (a >> lane) & 1u, inb = (bmask >> lane) & 1u;
    uint32_t u = a | bmask;
    if (base == (own0 & ~31)) u &= ~(3u << (own0 & 31));        // own0 is even: both own blocks lie in one word
    const bool sel = (u >> lane) & 1u;
    if (sel) dst[out + __popc(u & ((1u << lane) - 1u))] = kb | (ina ? (1 << 30) : 0) | (inb ? (int)(1u << 31) : 0);
    out += __popc(u);
  }
  __syncwarp();
  if (lane == 0) {
    if (out & 1) { dst[out] = dst[out - 1] & 0x3fffffff; }   // odd tail: second half of the last tile is nobody's
    clean_cnt[pair] = (out + 1) >> 1;
  }
}

// FP8: largest V block scale of every (batch, head); one warp each
__global__ void head_vmax_kernel(const float* __restrict__ v_scale, float* __restrict__ v_max, int bh_count, int nb) {
  const int bh = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (bh >= bh_count) return;
  float m = 0.0f;
  for (int j = lane; j < nb; j += 32) m = fmaxf(m, __ldg(v_scale + (int64_t)bh * nb + j));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) v_max[bh] = m;
}

__device__ __forceinline__ void pipe_tma_store_4d(const void* tmap, const void* smem_src, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
      ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}

// PAIR: 64-token blocks; a work item is a pair of query blocks, a tile two key blocks (see pair_lists_kernel).
// GATE (bf16, 128-token blocks, no window): the closing warpgroup of an item also computes the low-rank branch
// of its 128 query rows and writes O = O_s + g * r * RMSNorm(q~ C) instead of O_s: the item's Q tile is still in
// shared memory and its normalised output row in registers, so the separate pass that would read Q and O_s
// again and write O falls away.  The V ring gives up one slot for P_q and C of the current head.
template <bool FP8, bool WINDOW, bool PAIR, bool GATE = false, bool EPI = false>
__global__ void __launch_bounds__(EPI ? kEpiThreads : kPipeThreads, 1)
fwd_pipe_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                const __grid_constant__ CUtensorMap tmap_p, const PipeParams p) {
  static_assert(!GATE || (!FP8 && !WINDOW && !PAIR), "the fused gate epilogue exists for plain bf16 only");
  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* sQ = smem + kOffQ;
  unsigned char* sK = smem + kOffK;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kOffMisc);
  uint64_t* bar_q_full = bars + 0;     // [2]
  uint64_t* bar_q_free = bars + 2;     // [2] the item's output store has read the slot (or the item was empty)
  // An input tile is 128 rows x 128 channels: two 64-channel slabs of 16 KB in bf16, one slab in FP8, where the
  // same bytes hold rings twice as deep (the Q slots keep their 32 KB: the item's output is staged there).
  constexpr int kSlot = FP8 ? kTile / 2 : kTile;
  constexpr int RK = FP8 ? 4 : 2, RV = GATE ? 2 : (FP8 ? 6 : 3);    // (K 3 / V 2 measures the same)
  unsigned char* sV = sK + RK * kSlot;         // the V ring follows the K ring (5 x 32 KB between them)
  unsigned char* sP = sV + RV * kSlot;         // GATE: P_q of the current head (2 slabs of 8 KB), then C as bf16 (2 x 8 KB)
  unsigned char* sC = sP + 16384;
  uint64_t* bar_k_full = bars + 32;           // [RK]
  uint64_t* bar_k_free = bar_k_full + RK;     // [RK] S MMAs that read the slot are complete
  uint64_t* bar_v_full = bar_k_free + RK;     // [RV]
  uint64_t* bar_v_free = bar_v_full + RV;     // [RV] PV MMAs that read the slot are complete
  uint64_t* bar_cl = bars + 54;               // EPI [2], 128 arrivals: the sums of the warpgroup of the item's last tile are in Q slot i
  uint64_t* bar_gt = bars + 54;               // GATE [2]: the projection Q P_q^T of warpgroup g's closing is complete
  uint64_t* bar_gy = bars + 56;               // GATE [2]: y = q~ C is complete
  uint64_t* bar_pq = bars + 58;               // GATE [2]: P_q of a new head has landed
  uint64_t* bar_s_full = bars + 14;    // [2] S of a tile complete in S buffer (tile & 1)
  uint64_t* bar_s_free = bars + 16;    // [2] 128 arrivals: the warpgroup holds that S row in registers
  uint64_t* bar_p_full = bars + 18;    // [2] 128 arrivals: P written to P buffer (tile & 1)
  uint64_t* bar_pv_done = bars + 20;   // [2] PV of a tile complete: P buffer free again
  uint64_t* bar_o_free = bars + 22;    // 128 arrivals: the closing warpgroup has read O
  uint64_t* bar_tok = bars + 23;       // [2] 128 arrivals: warpgroup g has published its reference maxima
  uint64_t* bar_lsum = bars + 25;      // 128 arrivals: the non-closing warpgroup has published its row sums
  uint64_t* bar_lsum_ack = bars + 26;  // 128 arrivals: they have been read
  float* s_mref = reinterpret_cast<float*>(bars + 64);           // [2][128]
  float2* s_lsum = reinterpret_cast<float2*>(s_mref + 2 * 128);  // [128] (partial row sum, reference it is relative to)
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_lsum + 128);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  volatile int* s_gate_bh = s_abort + 1;      // GATE: (batch, head) whose P_q and C are in shared memory

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kTileTx = FP8 ? kTile / 2 : kTile;
  constexpr int kEnt = PAIR ? 2 : 1;              // list entries per tile
  constexpr int kKeyBlk = PAIR ? 64 : 128;        // tokens per key block

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_q_full + i, 1); mbar_init(bar_q_free + i, 1);
      mbar_init(bar_tok + i, 128);
      mbar_init(bar_s_full + i, 1); mbar_init(bar_s_free + i, 128);
      mbar_init(bar_p_full + i, 128); mbar_init(bar_pv_done + i, 1);
    }
    if constexpr (GATE) {
      for (int i = 0; i < 2; ++i) { mbar_init(bar_gt + i, 1); mbar_init(bar_gy + i, 1); mbar_init(bar_pq + i, 1); }
    } else if constexpr (EPI) {
      mbar_init(bar_cl, 128); mbar_init(bar_cl + 1, 128);
    }
    *s_gate_bh = -1;
    for (int i = 0; i < RK; ++i) { mbar_init(bar_k_full + i, 1); mbar_init(bar_k_free + i, 1); }
    for (int i = 0; i < RV; ++i) { mbar_init(bar_v_full + i, 1); mbar_init(bar_v_free + i, 1); }
    mbar_init(bar_o_free, 128); mbar_init(bar_lsum, 128); mbar_init(bar_lsum_ack, 128);
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
      tma_prefetch_desc(&tmap_q); tma_prefetch_desc(&tmap_k); tma_prefetch_desc(&tmap_v); tma_prefetch_desc(&tmap_o);
      if constexpr (GATE) tma_prefetch_desc(&tmap_p);
    }
    __syncwarp();
    tmem_alloc(s_tmem, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const uint32_t tmem_P = tmem + 2 * kPBLK;          // P buffer g at columns [256 + 64 g, +64)
  const uint32_t tmem_O = tmem + 3 * kPBLK;
  const bool dead = *s_abort != 0;
  const int first_item = blockIdx.x, item_step = gridDim.x;

  static_assert(!EPI || !GATE, "the gated variant closes its items in the softmax warpgroups");
  if constexpr (EPI) {
    if (warp < 4) reg_dec<kEpiCtrlRegs>();
    else if (warp >= 12) reg_dec<kEpiCloseRegs>();
  } else {
    if (warp < 4) reg_dec<kPipeCtrlRegs>();
  }
  if (dead) {
    // fall through to the teardown
  } else if (warp == 0 || warp == 3) {
    // ------------------------------------------------------------ TMA producers: warp 0 Q + the K ring, warp 3 the V ring
    // One thread each, walking the CTA's tile stream across item boundaries.  A producer only ever waits for
    // one thing, the release of the slot it fills next, so it sleeps in that barrier wait (a loop polling
    // several barriers with a back-off reacts to a freed slot up to a microsecond late, which is exposed
    // latency on a two-slot ring).  List entries and item counts are fetched one step ahead of their use.
    if (lane == 0) {
      const bool is_v = warp == 3;
      unsigned char* ring = is_v ? sV : sK;
      const CUtensorMap* map = is_v ? &tmap_v : &tmap_k;
      uint64_t* bar_full = is_v ? bar_v_full : bar_k_full;
      uint64_t* bar_free = is_v ? bar_v_free : bar_k_free;
      const int R = is_v ? RV : RK;
      int ord = 0, t = 0;                               // items seen, tiles loaded so far
      int item = first_item;
      int cnt = item < p.items ? __ldg(p.clean_cnt + item) : 0;
      int kb = item < p.items ? __ldg(p.clean_list + (int64_t)item * p.lstride) : 0;
      int kb2 = (PAIR && item < p.items) ? __ldg(p.clean_list + (int64_t)item * p.lstride + 1) : 0;
      bool ok = true;
      while (ok && item < p.items) {
        // the next item's count and first entries, needed when this item is done
        const int nxt = item + item_step;
        const int cnt_next = nxt < p.items ? __ldg(p.clean_cnt + nxt) : 0;
        const int kb_next = nxt < p.items ? __ldg(p.clean_list + (int64_t)nxt * p.lstride) : 0;
        const int kb2_next = (PAIR && nxt < p.items) ? __ldg(p.clean_list + (int64_t)nxt * p.lstride + 1) : 0;
        const int bh = item / p.nbq;
        const int hh = bh % p.H, bb = bh / p.H;
        if (!is_v) {
          const int qslot = ord & 1;
          if (cnt > 0) {
            if (ord >= 2) ok = mbar_wait(bar_q_free + qslot, ((ord >> 1) - 1) & 1, s_abort, p.status, 1);
            if (!ok) break;
            const int qb = item % p.nbq;
            mbar_expect_tx(bar_q_full + qslot, kTileTx);
            tma_load_4d(sQ + qslot * kTile, &tmap_q, bar_q_full + qslot, 0, qb * kPBLK, hh, bb);
            if constexpr (!FP8) tma_load_4d(sQ + qslot * kTile + kTile / 2, &tmap_q, bar_q_full + qslot, 64, qb * kPBLK, hh, bb);
          } else {
            mbar_arrive(bar_q_full + qslot);            // empty item: nothing to load, consumers still step through it
          }
        }
        for (int n = 0; ok && n < cnt; ++n, ++t) {
          const int slot = t % R;
          // the entries of the tile after this one (used one step later)
          int kb_n = 0, kb2_n = 0;
          if (n + 1 < cnt) {
            kb_n = __ldg(p.clean_list + (int64_t)item * p.lstride + (n + 1) * kEnt);
            if constexpr (PAIR) kb2_n = __ldg(p.clean_list + (int64_t)item * p.lstride + (n + 1) * kEnt + 1);
          }
          if (t >= R) ok = mbar_wait(bar_free + slot, ((t / R) - 1) & 1, s_abort, p.status, is_v ? 16 : 1);
          if (!ok) break;
          unsigned char* dst = ring + slot * kSlot;
          uint64_t* bar = bar_full + slot;
          mbar_expect_tx(bar, kTileTx);
          // one K or V tile: 128 key rows of one block, or 64 + 64 rows of the tile's two 64-token blocks
          if constexpr (PAIR) {
            const int r0 = (kb & 0x3fffffff) * 64, r1 = (kb2 & 0x3fffffff) * 64;
            tma_load_4d(dst, map, bar, 0, r0, hh, bb);
            tma_load_4d(dst + 8192, map, bar, 0, r1, hh, bb);
            if constexpr (!FP8) {
              tma_load_4d(dst + kTile / 2, map, bar, 64, r0, hh, bb);
              tma_load_4d(dst + kTile / 2 + 8192, map, bar, 64, r1, hh, bb);
            }
          } else {
            tma_load_4d(dst, map, bar, 0, kb * kPBLK, hh, bb);
            if constexpr (!FP8) tma_load_4d(dst + kTile / 2, map, bar, 64, kb * kPBLK, hh, bb);
          }
          kb = kb_n; kb2 = kb2_n;
        }
        item = nxt; ++ord;
        cnt = cnt_next; kb = kb_next; kb2 = kb2_next;
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- S issuer: S = Q K^T of the next tile
    if (lane == 0) {
      constexpr uint32_t idesc_qk = make_idesc(FP8 ? 0u : 1u, 128, kPBLK, false);
      int si = 0, s_item = first_item, s_n = 0, s_cnt = -1, s_t = 0;
      bool ok = true;
      while (ok && s_item < p.items) {
        if (s_cnt < 0) s_cnt = __ldg(p.clean_cnt + s_item);
        if (s_n >= s_cnt) {
          s_item += item_step; ++si; s_n = 0; s_cnt = -1;
          continue;
        }
        const int sbuf = s_t & 1, kslot = s_t % RK, qslot = si & 1;
        const uint64_t dQ = make_smem_desc_sw128(smem_u32(sQ + qslot * kTile), 16);
        const uint64_t dK = make_smem_desc_sw128(smem_u32(sK + kslot * kSlot), 16);
        const uint32_t q_lo = (uint32_t)dQ, q_hi = (uint32_t)(dQ >> 32), k_lo = (uint32_t)dK, k_hi = (uint32_t)(dK >> 32);
        // The product needs all three (its S buffer free, K landed, Q landed), so the thread sleeps in one barrier
        // wait after the other instead of polling them with a back-off: the K tile, which is waited for longest,
        // comes first; the others have normally happened by then.
        ok = mbar_wait(bar_k_full + kslot, (s_t / RK) & 1, s_abort, p.status, 2);
        if (ok && s_n == 0) ok = mbar_wait(bar_q_full + qslot, (si >> 1) & 1, s_abort, p.status, 17);
        if (ok && s_t >= 2) ok = mbar_wait(bar_s_free + sbuf, ((s_t >> 1) - 1) & 1, s_abort, p.status, 18);   // row of tile s_t - 2 is in registers
        if (!ok) break;
        {
          tc_fence_after();
          // 32 bytes of the channel dimension per MMA: 16 bf16 (8 MMAs over two slabs) or 32 E4M3 (4 MMAs)
#pragma unroll
          for (int sl = 0; sl < (FP8 ? 1 : 2); ++sl)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              mma_ss<FP8>(tmem + sbuf * kPBLK, make_desc(q_lo + ((sl * (kTile / 2) + kk * 32) >> 4), q_hi),
                          make_desc(k_lo + ((sl * (kTile / 2) + kk * 32) >> 4), k_hi), idesc_qk, (sl | kk) != 0 ? 1u : 0u);
          tc_commit(bar_s_full + sbuf);
          tc_commit(bar_k_free + kslot);
          ++s_n; ++s_t;
        }
      }
    }
  } else if (warp == 2) {
    // -------------------------------------------------------------- PV issuer: O += P V of the oldest pending tile
    // (its own warp on another scheduler: an issuing thread shares its scheduler with two softmax
    // warps that are almost always ready, and gets an issue slot only when they stall)
    if (lane == 0) {
      constexpr uint32_t idesc_pv = make_idesc(FP8 ? 0u : 1u, 128, kPD, true);
      constexpr int kPvSteps = FP8 ? 4 : 8;          // 32 bytes of P per row per MMA: 16 bf16 or 32 E4M3 keys
      int p_item = first_item, p_n = 0, p_cnt = -1, p_t = 0, p_nonempty = 0;
      bool ok = true;
      while (ok && p_item < p.items) {
        if (p_cnt < 0) p_cnt = __ldg(p.clean_cnt + p_item);
        if (p_n >= p_cnt) {
          if (p_cnt > 0) ++p_nonempty;
          p_item += item_step; p_n = 0; p_cnt = -1;
          continue;
        }
        const int pbuf = p_t & 1, vslot = p_t % RV;
        const uint64_t dV = make_smem_desc_sw128(smem_u32(sV + vslot * kSlot), kTile / 2);
        const uint32_t v_lo = (uint32_t)dV, v_hi = (uint32_t)(dV >> 32);
        // (see the S issuer) the V tile and the previous item's closer first, P, which arrives last, last
        ok = mbar_wait(bar_v_full + vslot, (p_t / RV) & 1, s_abort, p.status, 10);
        // first tile of an item only: O of the previous item must have been read by its closer
        if (ok && p_n == 0 && p_nonempty > 0) ok = mbar_wait(bar_o_free, (p_nonempty - 1) & 1, s_abort, p.status, 19);
        if (ok) ok = mbar_wait(bar_p_full + pbuf, (p_t >> 1) & 1, s_abort, p.status, 20);
        if (!ok) break;
        {
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < kPvSteps; ++kk)
            mma_ts<FP8>(tmem_O, tmem_P + pbuf * 64 + kk * 8, make_desc(v_lo + ((kk * (128 / kPvSteps) * 128) >> 4), v_hi),
                        idesc_pv, (p_n == 0 && kk == 0) ? 0u : 1u);
          tc_commit(bar_pv_done + pbuf);
          tc_commit(bar_v_free + vslot);
          ++p_n; ++p_t;
        }
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ----------------------------------------------------------------- softmax
    if constexpr (EPI) reg_inc<kEpiSoftmaxRegs>(); else reg_inc<kPipeSoftmaxRegs>();
    const int g = (warp >> 2) - 1;                    // warpgroup: takes the tiles with (global tile counter & 1) == g
    const int row = threadIdx.x & 127;                // query row inside the block = TMEM lane
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    constexpr float kLazy = FP8 ? kPipeFp8LazyLog2 : kPipeLazyLog2;
    float m_used = 0.0f, l = 0.0f;                    // reference maximum this warpgroup last used; its partial row sum
    int t = 0;                                        // global tile counter at the start of the item
    int nonempty = 0;                                 // non-empty items finished so far
    bool ok = true;
    int io = 0;
    int closings = 0, gate_loads = 0;                 // GATE: items this warpgroup has closed, heads it has staged (barrier phases)
    // Line-up of the warpgroup's 128 threads on a named barrier.  A hardware barrier has no time limit, so it
    // is fenced by the abort flag: no warp enters it once the flag is up, and a warp that leaves its loop
    // early arrives once on its way out, which releases the warps that were already inside (every other warp
    // either is inside or will see the flag and arrive as well: the 128 arrivals always come together).
    auto wg_line_up = [&](int) {
      if (*s_abort) return false;
      asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory");
      return true;
    };
    // GATE (a softmax warpgroup closes the item, lists are short): the thread that stores an item's output does not wait
    // until the copy has read the Q slot (about 1300 clocks, on the path to the closing warpgroup's next tile);
    // it releases the slot after its next tile, or, should the item after the next come first (its Q goes into
    // this very slot), before that.
    constexpr bool kDeferStoreWait = GATE;            // (elsewhere the extra test per tile costs more than the wait: lists are long, or FP8)
    int store_slot = -1, store_io = 0;                // row 0: Q slot whose output store is in flight, and its item
    auto store_flush = [&]() {
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      mbar_arrive(bar_q_free + store_slot);
      store_slot = -1;
    };
    for (int item = first_item; ok && item < p.items; item += item_step, ++io) {
      const int qslot = io & 1;
      const int cnt = __ldg(p.clean_cnt + item);
      if constexpr (kDeferStoreWait) {
        if (row == 0 && store_slot >= 0 && io >= store_io + 2) store_flush();
      }
      const int qb = item % p.nbq, bh = item / p.nbq;     // PAIR: qb counts pairs of 64-token query blocks
      const int h = bh % p.H, b = bh / p.H;
      const int q_row = qb * kPBLK + row;
      const bool row_valid = q_row < p.N;
      // keys this row may attend to: [klo, khi) (everything up to N without a causal window)
      int klo = 0, khi = p.N;
      if constexpr (WINDOW) {
        const int fi = min(q_row, p.N - 1) / p.frame_tokens;
        klo = max(fi - p.window + 1, 0) * p.frame_tokens;
        khi = (int)min((long long)(fi + 1) * p.frame_tokens, (long long)p.N);
      }
      if (cnt == 0) {
        if (g == 0) {
          // empty kept list: zero output, lse = -inf; release the item's Q slot
          ok = __all_sync(0xffffffffu, mbar_wait(bar_q_full + qslot, (io >> 1) & 1, s_abort, p.status, 3));
          if (!ok) break;
          if (row_valid) {
            __nv_bfloat16* orow = p.out + b * p.stride_b + h * p.stride_h + (int64_t)q_row * p.stride_n;
#pragma unroll
            for (int ch = 0; ch < kPD / 8; ++ch) reinterpret_cast<uint4*>(orow)[ch] = make_uint4(0u, 0u, 0u, 0u);
            if (p.lse) p.lse[(int64_t)bh * p.N + q_row] = -INFINITY;
          }
          if (row == 0) mbar_arrive(bar_q_free + qslot);
        }
        continue;
      }
      l = 0.0f;
      float q_sc = 1.0f, v_max = 1.0f;
      if constexpr (FP8) {
        q_sc = PAIR ? __ldg(p.q_scale + (int64_t)bh * p.nb + min(2 * qb + (row >> 6), p.nb - 1)) : __ldg(p.q_scale + item);
        v_max = __ldg(p.v_max + bh);
      }
      // This warpgroup's tiles are n0, n0 + 2, ...  List entries are fetched two of its tiles ahead and the FP8
      // scales of a tile one tile ahead, so that neither load (nor the two in a row, entry then scale) is waited
      // for inside the tile loop.
      const int n0 = (g ^ t) & 1;
      const int32_t* lst = p.clean_list + (int64_t)item * p.lstride;
      const float* ksc = FP8 ? p.k_scale + (int64_t)bh * p.nb : nullptr;
      const float* vsc = FP8 ? p.v_scale + (int64_t)bh * p.nb : nullptr;
      auto ld_ent = [&](int n, int e) { return n < cnt ? __ldg(lst + n * kEnt + e) : 0; };
      int e_cur0 = ld_ent(n0, 0), e_cur1 = PAIR ? ld_ent(n0, 1) : 0;
      int e_nx0 = ld_ent(n0 + 2, 0), e_nx1 = PAIR ? ld_ent(n0 + 2, 1) : 0;
      float ks_cur0 = 1.0f, vs_cur0 = 1.0f, ks_cur1 = 1.0f, vs_cur1 = 1.0f;
      int bv_cur = kKeyBlk, bv_cur1 = kKeyBlk;     // real tokens of the tile's key block(s) (bricks padded to whole blocks)
      if (p.blk_valid != nullptr) {
        bv_cur = __ldg(p.blk_valid + (e_cur0 & 0x3fffffff));
        if constexpr (PAIR) bv_cur1 = __ldg(p.blk_valid + (e_cur1 & 0x3fffffff));
      }
      if constexpr (FP8) {
        ks_cur0 = __ldg(ksc + (e_cur0 & 0x3fffffff));
        vs_cur0 = __ldg(vsc + (e_cur0 & 0x3fffffff));
        if constexpr (PAIR) {
          ks_cur1 = __ldg(ksc + (e_cur1 & 0x3fffffff));
          vs_cur1 = __ldg(vsc + (e_cur1 & 0x3fffffff));
        }
      }
      const float inv_vmax = 1.0f / v_max;
      for (int n = n0; ok && n < cnt; n += 2) {
        const int tt = t + n;
        const int buf = g;                          // (tt & 1) == g: this warpgroup's S and P buffers
        // the tile's key block(s); PAIR: two 64-token blocks, each with a flag per query block of the pair
        const int e0 = e_cur0, e1 = e_cur1;
        const float ks0 = ks_cur0, vs0 = vs_cur0, ks1 = ks_cur1, vs1 = vs_cur1;
        const int bv0 = bv_cur, bv1 = bv_cur1;
        if (p.blk_valid != nullptr) {
          bv_cur = __ldg(p.blk_valid + (e_nx0 & 0x3fffffff));
          if constexpr (PAIR) bv_cur1 = __ldg(p.blk_valid + (e_nx1 & 0x3fffffff));
        }
        // next tile of this warpgroup: its scales (its entries arrived a tile ago), and the entries of the one after
        if constexpr (FP8) {
          ks_cur0 = __ldg(ksc + (e_nx0 & 0x3fffffff));
          vs_cur0 = __ldg(vsc + (e_nx0 & 0x3fffffff));
          if constexpr (PAIR) {
            ks_cur1 = __ldg(ksc + (e_nx1 & 0x3fffffff));
            vs_cur1 = __ldg(vsc + (e_nx1 & 0x3fffffff));
          }
        }
        e_cur0 = e_nx0; e_cur1 = e_nx1;
        e_nx0 = ld_ent(n + 4, 0);
        if constexpr (PAIR) e_nx1 = ld_ent(n + 4, 1);
        int kb, kb1 = 0;
        bool mem0 = true, mem1 = true;
        if constexpr (PAIR) {
          kb = e0 & 0x3fffffff;
          kb1 = e1 & 0x3fffffff;
          mem0 = (((uint32_t)e0 >> (30 + (row >> 6))) & 1u) != 0u;
          mem1 = (((uint32_t)e1 >> (30 + (row >> 6))) & 1u) != 0u;
        } else {
          kb = e0;
        }
        float c = p.scale_log2;                      // logit -> log2 units
        float p_off = 0.0f;                          // log2 of the factor folded into P
        float c1 = c, p_off1 = 0.0f;                 // PAIR + FP8: the second key block of the tile has its own scales
        if constexpr (FP8) {
          c *= q_sc * ks0;
          p_off = kPipeFp8PScaleLog2 + log2f(vs0 * inv_vmax);
          if constexpr (PAIR) {
            c1 *= q_sc * ks1;
            p_off1 = kPipeFp8PScaleLog2 + log2f(vs1 * inv_vmax);
          }
        }
        // this row's valid columns: [c_lo, c_hi) of the tile, or (PAIR) [c_lo, c_hi) of its first 64 and
        // [c_lo1, c_hi1) of its second 64 columns (empty when the block is not in this query block's list)
        const int c_lo = klo - kb * kKeyBlk, c_hi = PAIR ? (mem0 ? min(khi - kb * 64, bv0) : 0) : min(khi - kb * kPBLK, bv0);
        const int c_lo1 = klo - kb1 * 64, c_hi1 = mem1 ? min(khi - kb1 * 64, bv1) : 0;
        ok = __all_sync(0xffffffffu, mbar_wait(bar_s_full + buf, (tt >> 1) & 1, s_abort, p.status, 4));
        if (!ok) break;
        tc_fence_after();
        const uint32_t tS = tmem + buf * kPBLK + lane_off;
        uint32_t sr[kPBLK];
#pragma unroll
        for (int ch = 0; ch < kPBLK / 32; ++ch) tmem_ld32(tS + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&sr[ch * 32]));
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(bar_s_free + buf);    // the S buffer can take the next-but-one tile
        if constexpr (PAIR) {
          if ((WINDOW && (c_lo > 0 || c_lo1 > 0)) || c_hi < 64 || c_hi1 < 64) {
#pragma unroll
            for (int i = 0; i < 64; ++i) {
              if ((WINDOW && i < c_lo) || i >= c_hi) sr[i] = 0xff800000u;
              if ((WINDOW && i < c_lo1) || i >= c_hi1) sr[64 + i] = 0xff800000u;
            }
          }
        } else if ((WINDOW && c_lo > 0) || c_hi < kPBLK) {   // ragged last key block / padding rows of a brick / keys outside the causal window get weight 0
          if (!WINDOW && c_hi >= kPBLK - 32) {                // a short tail (every tile of a padded brick layout): 32 tests, not 128
#pragma unroll
            for (int i = kPBLK - 32; i < kPBLK; ++i)
              if (i >= c_hi) sr[i] = 0xff800000u;
          } else {
#pragma unroll
            for (int i = 0; i < kPBLK; ++i)
              if ((WINDOW && i < c_lo) || i >= c_hi) sr[i] = 0xff800000u;
          }
        }
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]);
        float mx2 = __uint_as_float(sr[2]), mx3 = __uint_as_float(sr[3]);
#pragma unroll
        for (int i = 4; i < kPBLK; i += 8) {
          mx0 = fmax3(mx0, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
          mx1 = fmax3(mx1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
          if (i + 4 < kPBLK) {
            mx2 = fmax3(mx2, __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
            mx3 = fmax3(mx3, __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
          }
        }
        float m_tile = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * c;
        if constexpr (PAIR && FP8) {      // two logit scales in one tile: maxima of the two halves separately
          float ma = __uint_as_float(sr[0]), mb = __uint_as_float(sr[64]);
#pragma unroll
          for (int i = 1; i < 64; i += 2) {
            ma = fmax3(ma, __uint_as_float(sr[i]), __uint_as_float(sr[(i + 1) & 63]));
            mb = fmax3(mb, __uint_as_float(sr[64 + i]), __uint_as_float(sr[64 + ((i + 1) & 63)]));
          }
          m_tile = fmaxf(ma * c, mb * c1);
        }

        // reference maximum: token from the warpgroup of tile tt-1 (also orders the reuse of s_mref[g])
        if (tt > 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar_tok + (g ^ 1), ((tt - 1) >> 1) & 1, s_abort, p.status, 5));
          if (!ok) break;
        }
        float m_new;
        bool need = false;
        float alpha = 1.0f;
        if (n == 0) {
          m_new = m_tile;
        } else {
          const float m_prev = s_mref[(g ^ 1) * 128 + row];
          if (m_prev == -INFINITY) {
            m_new = m_tile;             // nothing accumulated for this row yet (all keys so far masked): O row and l are 0
          } else if (m_tile > m_prev + kLazy) {
            m_new = m_tile;
            alpha = fast_exp2(m_prev - m_tile);
            need = true;
          } else {
            m_new = m_prev;
          }
        }
        if (l != 0.0f && m_new != m_used) l *= fast_exp2(m_used - m_new);   // own partial sum to the new reference
        m_used = m_new;
        if (__any_sync(0xffffffffu, need)) {
          // Every PV issued so far must be complete before O is rescaled: the last one is tile tt-1's,
          // tracked by the other warpgroup's barrier.  A parity wait is only sound while the barrier is
          // at most one completion behind the one waited for, and the other warpgroup may not have
          // waited for PV of tile tt-3 yet; PVs complete in order, so PV of tile tt-2 (this warpgroup's
          // own barrier, whose previous completion it has already seen) is waited for first.
          if (tt >= 2) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + buf, ((tt >> 1) - 1) & 1, s_abort, p.status, 12));
            if (!ok) break;
          }
          ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + ((tt - 1) & 1), ((tt - 1) >> 1) & 1, s_abort, p.status, 6));
          if (!ok) break;
          tc_fence_after();
          const uint64_t a2 = pack_f32x2(alpha, alpha);
#pragma unroll 1
          for (int ch = 0; ch < kPD / 32; ++ch) {
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
          tc_wait_st();
          tc_fence_before();
        }
        s_mref[g * 128 + row] = m_used;
        mbar_arrive(bar_tok + g);

        // P = exp2(S*c - m) as bf16 into this warpgroup's P buffer
        const uint32_t tP = tmem_P + buf * 64 + lane_off;
        const float neg_m = m_used == -INFINITY ? 0.0f : p_off - m_used;     // a fully masked row: exp2(-inf) = 0, not NaN
        const float neg_m1 = m_used == -INFINITY ? 0.0f : p_off1 - m_used;
        const uint64_t c2a = pack_f32x2(c, c), nm2a = pack_f32x2(neg_m, neg_m);
        const uint64_t c2b = pack_f32x2(c1, c1), nm2b = pack_f32x2(neg_m1, neg_m1);
        uint64_t lsum0 = pack_f32x2(0.0f, 0.0f), lsum1 = lsum0;
        constexpr int kWords = FP8 ? 8 : 16;        // 32-bit words of P per 32 S columns
#pragma unroll
        for (int ch = 0; ch < kPBLK / 32; ++ch) {
          uint32_t w[kWords];
          float e[32];
          const bool second = PAIR && FP8 && ch >= 2;       // the tile's second key block: its own scales, its own sum
          const uint64_t c2 = second ? c2b : c2a, nm2 = second ? nm2b : nm2a;
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float2 x = unpack_f32x2(
                ffma2(pack_f32x2(__uint_as_float(sr[ch * 32 + i]), __uint_as_float(sr[ch * 32 + i + 1])), c2, nm2));
            e[i] = fast_exp2(x.x);
            e[i + 1] = fast_exp2(x.y);
            if ((PAIR && FP8) ? second : (((i >> 1) & 1) != 0)) lsum1 = fadd2(lsum1, pack_f32x2(e[i], e[i + 1]));
            else lsum0 = fadd2(lsum0, pack_f32x2(e[i], e[i + 1]));
          }
          if constexpr (FP8) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(e[4 * i], e[4 * i + 1]), __NV_SATFINITE, __NV_E4M3);
              const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(e[4 * i + 2], e[4 * i + 3]), __NV_SATFINITE, __NV_E4M3);
              w[i] = lo | (hi << 16);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(e[2 * i], e[2 * i + 1]);
              w[i] = *reinterpret_cast<const uint32_t*>(&h2);
            }
          }
          if (ch == 0 && tt >= 2) {
            // this warpgroup's P buffer is free once PV of tile tt-2 is complete (normally long ago)
            ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + buf, ((tt >> 1) - 1) & 1, s_abort, p.status, 11));
          }
          if constexpr (FP8) tmem_st8(tP + ch * 8, w);
          else tmem_st16(tP + ch * 16, w);
        }
        if constexpr (PAIR && FP8) {       // the row sum is kept without the factors folded into P, one per key block
          const float2 la = unpack_f32x2(lsum0), lb = unpack_f32x2(lsum1);
          l += (la.x + la.y) * fast_exp2(-p_off) + (lb.x + lb.y) * fast_exp2(-p_off1);
        } else {
          const float2 ls = unpack_f32x2(fadd2(lsum0, lsum1));
          if constexpr (FP8) l += (ls.x + ls.y) * fast_exp2(-p_off);
          else l += ls.x + ls.y;
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_full + buf);
        if constexpr (kDeferStoreWait) {
          if (row == 0 && store_slot >= 0) store_flush();
        }
      }
      if (!ok) break;

      // ------------------------------------------------------------ end of the item
      const int t_last = t + cnt - 1;
      if constexpr (EPI) {
        // The closing warpgroup (warps 12-15) finishes the item; the softmax warpgroups only leave it their
        // partial row sums and the reference they are relative to, and go on to the next item's tiles: the
        // warpgroup of the item's last tile in the first KB of the item's Q slot (it has read the last S, so every
        // S product of the item is complete and Q is dead), the other one in s_lsum.
        if ((t_last & 1) != g) {
          if (nonempty > 0) {
            ok = __all_sync(0xffffffffu, mbar_wait(bar_lsum_ack, (nonempty - 1) & 1, s_abort, p.status, 7));
            if (!ok) break;
          }
          s_lsum[row] = make_float2(l, m_used);
          mbar_arrive(bar_lsum);
        } else {
          reinterpret_cast<float2*>(sQ + qslot * kTile)[row] = make_float2(l, m_used);
          mbar_arrive(bar_cl + qslot);
        }
      } else if ((t_last & 1) != g) {
        // not the closer: hand the partial row sum over (after the previous hand-over was read)
        if (nonempty > 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(bar_lsum_ack, (nonempty - 1) & 1, s_abort, p.status, 7));
          if (!ok) break;
        }
        s_lsum[row] = make_float2(l, m_used);
        mbar_arrive(bar_lsum);
        // The two hand-over barriers are waited on by whichever warpgroup closes (or does not close) the
        // next item, with a phase parity counted in items; that is only sound if no thread of this
        // warpgroup runs ahead while the phase its own warpgroup completes is still open (items of one
        // or two tiles make that possible).  So the warpgroup lines up after arriving.
        ok = wg_line_up(13);
        if (!ok) break;
      } else {
        ok = __all_sync(0xffffffffu, mbar_wait(bar_lsum, nonempty & 1, s_abort, p.status, 8));
        if (!ok) break;
        const float2 other = s_lsum[row];
        mbar_arrive(bar_lsum_ack);
        ok = wg_line_up(14);                                            // see the note at the hand-over above
        if (!ok) break;
        if (other.x != 0.0f) l += other.x * fast_exp2(other.y - m_used);
        ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + (t_last & 1), (t_last >> 1) & 1, s_abort, p.status, 9));
        if (!ok) break;
        tc_fence_after();
        // normalised O row as bf16 into the item's Q slot (all S MMAs of the item are complete), 128-byte swizzle
        float inv = l > 0.0f ? 1.0f / l : 0.0f;           // no admissible key at all: zero row, lse = -inf
        if constexpr (FP8) inv *= v_max * 0.0625f;        // undo the 2^4 / max s_v folded into P
        unsigned char* slot = sQ + qslot * kTile;
        if constexpr (GATE) {
          // ---- P_q and C of this (batch, head), if another head's are in shared memory (the product that read them
          // last is complete: its warpgroup released O only after reading y)
          if (*s_gate_bh != bh) {
            if (row == 0) {
              mbar_expect_tx(bar_pq + g, 16384);
              tma_load_4d(sP, &tmap_p, bar_pq + g, 0, 0, h, 0);
              tma_load_4d(sP + 8192, &tmap_p, bar_pq + g, 64, 0, h, 0);
            }
            const int a = row >> 1, half = row & 1;      // thread j converts row a, columns [64 half, +64) of the fp32 state
            const float* src = p.state + ((int64_t)bh * kCompRank + a) * kPD + half * 64;
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
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            ok = __all_sync(0xffffffffu, mbar_wait(bar_pq + g, gate_loads & 1, s_abort, p.status, 21));
            ++gate_loads;
            if (ok) ok = wg_line_up(22);
            if (!ok) break;
            if (row == 0) *s_gate_bh = bh;
          }
          // ---- T = Q P_q^T into this warpgroup's P buffer (64 fp32 columns; its last P has been consumed)
          const uint32_t tT = tmem_P + g * 64;
          if (row == 0) {
            tc_fence_after();
            const uint64_t dX = make_smem_desc_sw128(smem_u32(slot), 16), dP = make_smem_desc_sw128(smem_u32(sP), 16);
            const uint32_t x_lo = (uint32_t)dX, x_hi = (uint32_t)(dX >> 32), p_lo = (uint32_t)dP, p_hi = (uint32_t)(dP >> 32);
            constexpr uint32_t idesc_t = make_idesc(1u, 128, kCompRank, false);
#pragma unroll
            for (int sl = 0; sl < 2; ++sl)
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                mma_ss<false>(tT, make_desc(x_lo + ((sl * 16384 + kk * 32) >> 4), x_hi),
                              make_desc(p_lo + ((sl * 8192 + kk * 32) >> 4), p_hi), idesc_t, (sl | kk) != 0 ? 1u : 0u);
            tc_commit(bar_gt + g);
          }
          // the row's rotary factors and gate value arrive under the wait for T
          float2 cs[kCompRank / 2];
          {
            const int token = min(q_row, p.N - 1);
            const int x = token % p.rope.Wg, yy = token / p.rope.Wg;
            const int y = yy % p.rope.Hg, tt = yy / p.rope.Hg;
            const float2* row_t = p.rope_table + tt * (kCompRank / 2);
            const float2* row_y = p.rope_table + (p.rope.T + y) * (kCompRank / 2);
            const float2* row_x = p.rope_table + (p.rope.T + p.rope.Hg + x) * (kCompRank / 2);
#pragma unroll
            for (int m = 0; m < kCompRank / 2; ++m) {
              const int ax = p.rope.axis[m];
              cs[m] = __ldg((ax == 0 ? row_t : (ax == 1 ? row_y : row_x)) + m);
            }
          }
          const float gte = row_valid ? __ldg(p.gate + (int64_t)bh * p.N + q_row) : 0.0f;
          ok = __all_sync(0xffffffffu, mbar_wait(bar_gt + g, closings & 1, s_abort, p.status, 23));
          if (!ok) break;
          tc_fence_after();
          // ---- q~ = R(p) silu(T) as bf16 over the first 32 columns of T (a thread only touches its own row)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t r[32];
            tmem_ld32(tT + lane_off + half * 32, r);
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
            tmem_st16(tT + lane_off + half * 16, w);
          }
          tc_wait_st();
          // ---- the O_s row, normalised and rounded to bf16, into registers; the sum of its squares for r_i
          uint32_t opk[kPD / 2];
          float so = 0.0f;
#pragma unroll
          for (int ch = 0; ch < kPD / 32; ++ch) {
            uint32_t r[32];
            tmem_ld32(tmem_O + lane_off + ch * 32, r);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[2 * j]) * inv, __uint_as_float(r[2 * j + 1]) * inv);
              opk[ch * 16 + j] = *reinterpret_cast<const uint32_t*>(&h2);
              const float2 f = __bfloat1622float2(h2);
              so = fmaf(f.x, f.x, fmaf(f.y, f.y, so));
            }
          }
          tc_fence_before();
          ok = wg_line_up(24);
          if (!ok) break;
          // ---- y = q~ C over the O columns (O_s is in registers): A = q~ from TMEM, B = C, d contiguous
          if (row == 0) {
            tc_fence_after();
            const uint64_t dC = make_smem_desc_sw128(smem_u32(sC), 8192);
            const uint32_t c_lo = (uint32_t)dC, c_hi = (uint32_t)(dC >> 32);
            constexpr uint32_t idesc_y = make_idesc(1u, 128, kPD, true);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              mma_ts<false>(tmem_O, tT + kk * 8, make_desc(c_lo + ((kk * 2048) >> 4), c_hi), idesc_y, kk != 0 ? 1u : 0u);
            tc_commit(bar_gy + g);
          }
          ok = __all_sync(0xffffffffu, mbar_wait(bar_gy + g, closings & 1, s_abort, p.status, 25));
          ++closings;
          if (!ok) break;
          tc_fence_after();
          // ---- two passes over y: its mean square, then O = O_s + g * r * y / rms(y) into the Q slot
          float ss = 0.0f;
#pragma unroll
          for (int ch = 0; ch < kPD / 32; ch += 2) {
            uint32_t r[32], r2[32];
            tmem_ld32(tmem_O + lane_off + ch * 32, r);
            tmem_ld32(tmem_O + lane_off + ch * 32 + 32, r2);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) ss = fmaf(__uint_as_float(r[j]), __uint_as_float(r[j]), ss);
#pragma unroll
            for (int j = 0; j < 32; ++j) ss = fmaf(__uint_as_float(r2[j]), __uint_as_float(r2[j]), ss);
          }
          const float coef = gte * sqrtf(so * (1.0f / kPD)) * rsqrtf(ss * (1.0f / kPD) + p.eps);
#pragma unroll
          for (int ch = 0; ch < kPD / 32; ++ch) {
            uint32_t r[32];
            tmem_ld32(tmem_O + lane_off + ch * 32, r);
            tc_wait_ld();
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
              uint32_t ww[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&opk[ch * 16 + cc * 4 + j]));
                const __nv_bfloat162 o2 = __floats2bfloat162_rn(fmaf(coef, __uint_as_float(r[8 * cc + 2 * j]), f.x),
                                                                fmaf(coef, __uint_as_float(r[8 * cc + 2 * j + 1]), f.y));
                ww[j] = *reinterpret_cast<const uint32_t*>(&o2);
              }
              *reinterpret_cast<uint4*>(slot + (ch >> 1) * (kTile / 2) + row * 128 + ((((ch & 1) * 4 + cc) ^ (row & 7)) << 4)) =
                  make_uint4(ww[0], ww[1], ww[2], ww[3]);
            }
          }
        } else {
#pragma unroll 1
        for (int ch = 0; ch < kPD / 32; ++ch) {
          uint32_t r[32];
          tmem_ld32(tmem_O + lane_off + ch * 32, r);
          tc_wait_ld();
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            uint32_t ww[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[8 * cc + 2 * j]) * inv,
                                                              __uint_as_float(r[8 * cc + 2 * j + 1]) * inv);
              ww[j] = *reinterpret_cast<const uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(slot + (ch >> 1) * (kTile / 2) + row * 128 + ((((ch & 1) * 4 + cc) ^ (row & 7)) << 4)) =
                make_uint4(ww[0], ww[1], ww[2], ww[3]);
          }
        }
        }
        tc_fence_before();
        mbar_arrive(bar_o_free);
        if (row_valid && p.lse) p.lse[(int64_t)bh * p.N + q_row] = (m_used + log2f(l)) * 0.6931471805599453f;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        ok = wg_line_up(15);
        if (!ok) break;
        if (row == 0) {
          pipe_tma_store_4d(&tmap_o, slot, 0, qb * kPBLK, h, b);
          pipe_tma_store_4d(&tmap_o, slot + kTile / 2, 64, qb * kPBLK, h, b);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          store_slot = qslot; store_io = io;
          if constexpr (!kDeferStoreWait) store_flush();
        }
      }
      t += cnt;
      ++nonempty;
    }
    if (!ok) asm volatile("bar.arrive %0, 128;" ::"r"(1 + g) : "memory");   // see wg_line_up
    if (row == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  else if (EPI && warp >= 12) {
    // ----------------------------------------------------------------- closing warpgroup (EPI variants)
    // Walks the CTA's items in order.  For each: the two partial row sums, the last PV, then the normalised O
    // row as bf16 into the item's Q slot, O back to the PV issuer, lse, one TMA store, the Q slot back to the
    // producer.  Nothing here is on the softmax warpgroups' path.
    const int row = threadIdx.x & 127;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    auto line_up = [&]() {
      if (*s_abort) return false;
      asm volatile("bar.sync 3, 128;" ::: "memory");
      return true;
    };
    int t = 0, nonempty = 0, io = 0;
    int slot_use[2] = {0, 0};                         // non-empty items that have used Q slot i
    bool ok = true;
    for (int item = first_item; ok && item < p.items; item += item_step, ++io) {
      const int cnt = __ldg(p.clean_cnt + item);
      if (cnt == 0) continue;                          // warpgroup 0 writes the zero rows of an empty list
      const int qslot = io & 1;
      const int qb = item % p.nbq, bh = item / p.nbq;
      const int h = bh % p.H, b = bh / p.H;
      const int q_row = qb * kPBLK + row;
      const bool row_valid = q_row < p.N;
      const int t_last = t + cnt - 1;
      unsigned char* slot = sQ + qslot * kTile;
      float v_max = 1.0f;
      if constexpr (FP8) v_max = __ldg(p.v_max + bh);
      // the slot's barrier completes once per non-empty item that uses the slot; this item's Q could only be
      // loaded after the previous user's output had left, so the wait is never more than one phase behind
      ok = __all_sync(0xffffffffu, mbar_wait(bar_cl + qslot, slot_use[qslot] & 1, s_abort, p.status, 8));
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_lsum, nonempty & 1, s_abort, p.status, 27));
      if (!ok) break;
      const float2 mine = reinterpret_cast<const float2*>(slot)[row];
      const float2 other = s_lsum[row];
      mbar_arrive(bar_lsum_ack);
      ++slot_use[qslot];
      float l = mine.x;
      const float m_used = mine.y;
      if (other.x != 0.0f) l += other.x * fast_exp2(other.y - m_used);
      ok = line_up();                                  // every row's sums are read before O rows overwrite them
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar_pv_done + (t_last & 1), (t_last >> 1) & 1, s_abort, p.status, 9));
      if (!ok) break;
      tc_fence_after();
      float inv = l > 0.0f ? 1.0f / l : 0.0f;          // no admissible key at all: zero row, lse = -inf
      if constexpr (FP8) inv *= v_max * 0.0625f;       // undo the 2^4 / max s_v folded into P
      // (16 columns at a time: this warpgroup runs on 40 registers, and what it spills goes to an L1 that the
      // shared-memory carve-out leaves very small)
#pragma unroll 1
      for (int ch = 0; ch < kPD / 16; ++ch) {
        uint32_t r[16];
        tmem_ld16(tmem_O + lane_off + ch * 16, r);
        tc_wait_ld();
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          uint32_t ww[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[8 * cc + 2 * j]) * inv,
                                                            __uint_as_float(r[8 * cc + 2 * j + 1]) * inv);
            ww[j] = *reinterpret_cast<const uint32_t*>(&h2);
          }
          *reinterpret_cast<uint4*>(slot + (ch >> 2) * (kTile / 2) + row * 128 + ((((ch & 3) * 2 + cc) ^ (row & 7)) << 4)) =
              make_uint4(ww[0], ww[1], ww[2], ww[3]);
        }
      }
      tc_fence_before();
      mbar_arrive(bar_o_free);
      if (row_valid && p.lse) p.lse[(int64_t)bh * p.N + q_row] = (m_used + log2f(l)) * 0.6931471805599453f;
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      ok = line_up();
      if (!ok) break;
      if (row == 0) {
        pipe_tma_store_4d(&tmap_o, slot, 0, qb * kPBLK, h, b);
        pipe_tma_store_4d(&tmap_o, slot + kTile / 2, 64, qb * kPBLK, h, b);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        mbar_arrive(bar_q_free + qslot);
      }
      t += cnt;
      ++nonempty;
    }
    if (!ok) asm volatile("bar.arrive 3, 128;" ::: "memory");
    if (row == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
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
// items (query blocks, or pairs of 64-token query blocks) per (batch, head), and list entries per item
static void pipe_geometry(const sparkattn_shape_t& s, int kmax, int* nbq, int* lstride) {
  const int nb = (s.N + s.block - 1) / s.block;
  const bool pair = s.block == 64;
  *nbq = pair ? (nb + 1) / 2 : nb;
  *lstride = pair ? 2 * kmax : kmax;
}

bool fwd_pipe_supported(const sparkattn_shape_t& s) {
  if (s.d != 128) return false;
  if (s.block == 128) return true;
  return s.block == 64 && (s.N + 63) / 64 <= kPairMaxBlocks;
}

size_t fwd_pipe_workspace_bytes(const sparkattn_shape_t& s, int kmax) {
  int nbq, lstride;
  pipe_geometry(s, kmax, &nbq, &lstride);
  const size_t items = (size_t)s.B * s.H * nbq;
  // header | tiles per item | compacted (merged) lists | FP8: largest V scale per (batch, head)
  return kWorkspaceHeaderBytes + (items * 4 + 255) / 256 * 256 + (items * (size_t)lstride * 4 + 255) / 256 * 256 +
         (size_t)s.B * s.H * 4;
}

bool fwd_pipe_gated_supported(const sparkattn_shape_t& s) { return s.d == 128 && s.block == 128; }

// ... | rotary table of the fused compensation epilogue
size_t fwd_pipe_gated_workspace_bytes(const sparkattn_shape_t& s, int kmax, const int32_t* grid) {
  return (fwd_pipe_workspace_bytes(s, kmax) + 255) / 256 * 256 + rope_table_bytes(grid);
}

// the compensation branch's operands of the fused epilogue (device pointers except grid / axis / freq)
struct PipeGateArgs {
  const void* pq;
  const int32_t* grid;
  const int32_t* axis;
  const float* freq;
  const float* state;
  const float* gate;
  float eps;
};

static int launch_pipe(const sparkattn_shape_t& s, bool fp8, const void* q, const void* k, const void* v,
                       const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                       const int32_t* kept_cnt, int kmax, int frame_tokens, int window, const int32_t* block_valid,
                       void* out, float* lse, void* workspace, const PipeGateArgs* ga, cudaStream_t stream);

int launch_fwd_pipe(const sparkattn_shape_t& s, bool fp8, const void* q, const void* k, const void* v,
                    const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                    const int32_t* kept_cnt, int kmax, int frame_tokens, int window, const int32_t* block_valid,
                    void* out, float* lse, void* workspace, cudaStream_t stream) {
  return launch_pipe(s, fp8, q, k, v, q_scale, k_scale, v_scale, kept_idx, kept_cnt, kmax, frame_tokens, window,
                     block_valid, out, lse, workspace, nullptr, stream);
}

int launch_fwd_pipe_gated(const sparkattn_shape_t& s, const void* q, const void* k, const void* v,
                          const int32_t* kept_idx, const int32_t* kept_cnt, int kmax, const void* pq,
                          const int32_t* grid, const int32_t* axis, const float* freq, const float* state,
                          const float* gate, float eps, void* out, float* lse, void* workspace, cudaStream_t stream) {
  const PipeGateArgs ga{pq, grid, axis, freq, state, gate, eps};
  return launch_pipe(s, false, q, k, v, nullptr, nullptr, nullptr, kept_idx, kept_cnt, kmax, 0, 0, nullptr, out, lse,
                     workspace, &ga, stream);
}

static int launch_pipe(const sparkattn_shape_t& s, bool fp8, const void* q, const void* k, const void* v,
                       const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                       const int32_t* kept_cnt, int kmax, int frame_tokens, int window, const int32_t* block_valid,
                       void* out, float* lse, void* workspace, const PipeGateArgs* ga, cudaStream_t stream) {
  CUtensorMap mq, mk, mv, mo, mp;
  int rc;
  const int elt = fp8 ? 1 : 2;
  const bool pair = s.block == 64;
  if ((rc = make_token_map(&mq, q, elt, s, kPBLK)) != SPARKATTN_OK) return rc;
  if ((rc = make_token_map(&mk, k, elt, s, pair ? 64 : kPBLK)) != SPARKATTN_OK) return rc;
  if ((rc = make_token_map(&mv, v, elt, s, pair ? 64 : kPBLK)) != SPARKATTN_OK) return rc;
  if ((rc = make_token_map(&mo, out, 2, s, kPBLK)) != SPARKATTN_OK) return rc;
  mp = mo;                                           // never read without the fused epilogue
  if (ga) {
    const uint64_t dims[4] = {(uint64_t)kPD, (uint64_t)kCompRank, (uint64_t)s.H, 1};
    const uint64_t strides[3] = {(uint64_t)kPD, (uint64_t)kCompRank * kPD, (uint64_t)s.H * kCompRank * kPD};
    if ((rc = make_slab_map(&mp, ga->pq, 2, dims, strides, kCompRank)) != SPARKATTN_OK) return rc;
  }
  const int nb = (s.N + s.block - 1) / s.block;
  int nbq, lstride;
  pipe_geometry(s, kmax, &nbq, &lstride);
  const long long items = (long long)s.B * s.H * nbq;
  if (items > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  char* base = static_cast<char*>(workspace);
  int32_t* clean_cnt = reinterpret_cast<int32_t*>(base + kWorkspaceHeaderBytes);
  int32_t* clean_list = reinterpret_cast<int32_t*>(base + kWorkspaceHeaderBytes + ((size_t)items * 4 + 255) / 256 * 256);
  float* v_max = reinterpret_cast<float*>(base + kWorkspaceHeaderBytes + ((size_t)items * 4 + 255) / 256 * 256 +
                                          ((size_t)items * lstride * 4 + 255) / 256 * 256);
  PipeParams prm{};
  prm.clean_cnt = clean_cnt;
  prm.clean_list = clean_list;
  prm.q_scale = q_scale; prm.k_scale = k_scale; prm.v_scale = v_scale; prm.v_max = v_max;
  prm.out = static_cast<__nv_bfloat16*>(out);
  prm.lse = lse;
  prm.status = static_cast<int32_t*>(workspace);
  prm.H = s.H; prm.N = s.N; prm.nb = nb; prm.items = (int)items; prm.nbq = nbq; prm.lstride = lstride;
  prm.frame_tokens = frame_tokens; prm.window = window;
  prm.blk_valid = block_valid;
  prm.stride_b = s.stride_b; prm.stride_h = s.stride_h; prm.stride_n = s.stride_n;
  const float sc = s.softmax_scale > 0.0f ? s.softmax_scale : 1.0f / sqrtf((float)s.d);
  prm.scale_log2 = sc * 1.4426950408889634f;
  const int sm_count = current_sm_count();
  if (sm_count < 1) return SPARKATTN_E_CUDA;
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  if (ga) {
    for (int m = 0; m < kCompRank / 2; ++m) { prm.rope.axis[m] = ga->axis[m]; prm.rope.freq[m] = ga->freq[m]; }
    prm.rope.T = ga->grid[0]; prm.rope.Hg = ga->grid[1]; prm.rope.Wg = ga->grid[2];
    float2* table = reinterpret_cast<float2*>(base + (fwd_pipe_workspace_bytes(s, kmax) + 255) / 256 * 256);
    launch_rope_table(prm.rope, table, stream);
    prm.rope_table = table;
    prm.state = ga->state; prm.gate = ga->gate; prm.eps = ga->eps;
  }
  if (pair) {
    const size_t bits = (size_t)kPairWarps * 2 * ((nb + 31) / 32) * sizeof(uint32_t);
    pair_lists_kernel<<<(unsigned)((items + kPairWarps - 1) / kPairWarps), kPairWarps * 32, bits, stream>>>(
        kept_idx, kept_cnt, clean_cnt, clean_list, (int)items, nb, nbq, kmax, prm.status);
  } else {
    compact_lists_kernel<<<(unsigned)((items + 7) / 8), 256, 0, stream>>>(kept_idx, kept_cnt, clean_cnt, clean_list,
                                                                        (int)items, nb, kmax, prm.status);
  }
  if (fp8) head_vmax_kernel<<<(unsigned)((s.B * s.H + 7) / 8), 256, 0, stream>>>(v_scale, v_max, s.B * s.H, nb);
  const bool win = frame_tokens > 0;
  auto kern = pair ? (fp8 ? (win ? fwd_pipe_kernel<true, true, true> : fwd_pipe_kernel<true, false, true>)
                          : (win ? fwd_pipe_kernel<false, true, true> : fwd_pipe_kernel<false, false, true>))
                   : (fp8 ? (win ? fwd_pipe_kernel<true, true, false> : fwd_pipe_kernel<true, false, false>)
                          : (win ? fwd_pipe_kernel<false, true, false> : fwd_pipe_kernel<false, false, false>));
  // short lists: the variant with a closing warpgroup (it takes the item boundary off the softmax warpgroups: 2.6 %
  // bf16 / 1 % FP8 at 18 tiles per item, 6-8 % at 6; but its tile loop is 3 % slower, and the two are level near 60
  // tiles per item)
  const bool epi = !ga && kmax <= kEpiMaxKept;
  if (epi && !fp8)
    kern = pair ? (win ? fwd_pipe_kernel<false, true, true, false, true> : fwd_pipe_kernel<false, false, true, false, true>)
                : (win ? fwd_pipe_kernel<false, true, false, false, true> : fwd_pipe_kernel<false, false, false, false, true>);
  if (epi && fp8)
    kern = pair ? (win ? fwd_pipe_kernel<true, true, true, false, true> : fwd_pipe_kernel<true, false, true, false, true>)
                : (win ? fwd_pipe_kernel<true, true, false, false, true> : fwd_pipe_kernel<true, false, false, false, true>);
  if (ga) kern = fwd_pipe_kernel<false, false, false, true>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kPipeSmem) != cudaSuccess)
    return SPARKATTN_E_CUDA;
  const unsigned grid = (unsigned)(items < sm_count ? items : sm_count);
  kern<<<grid, epi ? kEpiThreads : kPipeThreads, kPipeSmem, stream>>>(mq, mk, mv, mo, mp, prm);
  return cudaGetLastError() == cudaSuccess ? SPARKATTN_OK : SPARKATTN_E_CUDA;
}

}  // namespace sparkattn
