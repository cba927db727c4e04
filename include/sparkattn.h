/*
 * sparkattn -- block-sparse attention for long video-DiT token sequences on
 * NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes, no framework types.
 *
 * The library implements the sparse branch O_s = A_M(Q, K, V) of the paper's
 * compensated sparse attention (Sec. 2, "Block sparsity" and "Compensated
 * sparse attention"; Sec. 4.1): the attention matrix is cut into contiguous
 * query-block x key-block tiles, a selector keeps a fraction 1 - s of the key
 * blocks for every query block, and exact softmax attention
 * softmax(Q K^T / sqrt(d)) V is evaluated over the kept tiles only.
 *
 * Three device entry points make up the path:
 *   sparkattn_select     pooled block scores + top-k -> kept-block index lists
 *   sparkattn_quant_fp8  per-(head, token-block) absmax scale + E4M3 encode
 *   sparkattn_fwd        block-sparse flash-attention forward (bf16 or FP8)
 * plus one host-buffer convenience call that chains them with the copies, and
 * the low-rank compensation branch with the gate fusion that completes the
 * paper's attention module (sparkattn_comp_state, sparkattn_comp_apply).
 *
 * Conventions shared by all calls
 *   - Every data pointer is DEVICE memory owned by the caller unless a
 *     parameter name ends in `_host`.  The library allocates no device
 *     memory and keeps no pointer after the call returns.  What it does keep
 *     between calls, per device: two copy streams that
 *     sparkattn_attention_host creates on first use, the fixed scratch array
 *     of sparkattn_select_noalloc with its cached address, and the SM count.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream) and return without synchronising,
 *     except sparkattn_read_status and sparkattn_attention_host.
 *   - Tensors are [B, H, N, d] with d contiguous; strides are in elements.
 *   - Tokens are cut into nb = ceil(N / block) contiguous blocks; the last
 *     block may be ragged.  Rows >= N are never read as data or written.
 *   - Return value: SPARKATTN_OK (0) or a negative sparkattn_status code.
 *     Argument errors are detected on the host before anything is enqueued.
 *     Errors found on the device (a kept index outside [0, nb), a wait that
 *     ran out) are recorded in the first word of the caller's workspace and
 *     read back with sparkattn_read_status; the kernel skips the offending
 *     tile and still terminates.
 *   - Same inputs give bitwise identical outputs (no atomics on data, fixed
 *     reduction order).
 */
#ifndef SPARKATTN_H_
#define SPARKATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPARKATTN_VERSION 1

typedef enum {
  SPARKATTN_OK = 0,
  SPARKATTN_E_INVALID_ARG = -1,       /* NULL pointer, non-positive size, topk/kmax out of range      */
  SPARKATTN_E_UNSUPPORTED_SHAPE = -2, /* (d, block) not one of (64,64), (128,64), (128,128); nb too large */
  SPARKATTN_E_MISALIGNED = -3,        /* pointer not 16-byte aligned or stride * elem not 16-byte mult. */
  SPARKATTN_E_WORKSPACE_TOO_SMALL = -4,
  SPARKATTN_E_CUDA = -5,              /* launch or driver error; cudaGetLastError has the detail       */
  SPARKATTN_E_DEVICE_TIMEOUT = -6,    /* a bounded device-side wait expired (device status word)       */
  SPARKATTN_E_BAD_INDEX = -7,         /* a kept block index outside [0, nb) (device status word)       */
  SPARKATTN_E_NO_DEVICE = -8          /* no CUDA device / driver entry point unavailable               */
} sparkattn_status;

typedef enum { SPARKATTN_BF16 = 0, SPARKATTN_FP8_E4M3 = 1 } sparkattn_dtype;

/* Problem shape.  Caller fills it; the library reads it during the call only. */
typedef struct {
  uint32_t struct_size; /* sizeof(sparkattn_shape_t)                                   */
  uint32_t version;     /* SPARKATTN_VERSION                                           */
  int32_t B, H, N, d;   /* batch, heads (queries and keys share them), tokens, head dim */
  int32_t block;        /* tokens per query block = tokens per key block               */
  int32_t reserved;     /* must be 0                                                   */
  int64_t stride_b, stride_h, stride_n; /* element strides of [B,H,N,d]; d has stride 1 */
  float softmax_scale;  /* 0 selects 1/sqrt(d) (the paper's dense attention formula)   */
  uint32_t pad;         /* must be 0                                                   */
} sparkattn_shape_t;

int sparkattn_version(void);
const char* sparkattn_status_string(int status);

/* Bytes of device workspace a call needs.  which: 0 = sparkattn_select (pass
 * topk), 1 = sparkattn_fwd (pass kmax: for d = 128 the forward keeps a
 * range-checked copy of the kept lists (64-token blocks: the merged lists of
 * every pair of adjacent query blocks) and one scale per head behind the
 * status words, about 4 * B * H * nb * (kmax + 1) bytes either way; 256 bytes
 * for d = 64), 2 = sparkattn_gather_tokens (256).  Returns 0 for an invalid
 * shape or, for 0 and 1, a non-positive topk / kmax. */
size_t sparkattn_workspace_bytes(const sparkattn_shape_t* shape, int32_t which, int32_t topk_or_kmax);

/*
 * Block selection (the selector M_phi of Sec. 2 / Sec. 4.1; the paper lists
 * kinds of selectors, top-k over per-block scores among them, without fixing
 * a rule, so the rule is:)
 *   1. pooled sum over the valid tokens of a block, fp32, ascending token order
 *   2. pooled mean = sum / n_valid (IEEE fp32 divide)
 *   3. score(i, j) = fmaf chain over channels c ascending of pq[i,c] * pk[j,c]
 *   4. keep the `topk` key blocks first under (score descending, index ascending)
 *   5. write them in ascending index order.
 * Selection always reads the bf16 Q and K (Sec. 4.3 keeps mask selection in BF16).
 *
 * q_bf16, k_bf16 : in,  bf16 [B,H,N,d] with the strides of `shape`
 * topk           : in,  1 .. nb
 * kept_idx       : out, int32 [B,H,nb,topk] contiguous
 * kept_cnt       : out, int32 [B,H,nb] (every entry = topk); may be NULL
 * workspace      : scratch of >= sparkattn_workspace_bytes(shape, 0, topk) bytes,
 *                  256-byte aligned; its first word is the device status.
 */
int sparkattn_select(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                     int32_t* kept_idx, int32_t* kept_cnt, void* workspace, size_t workspace_bytes,
                     void* cuda_stream);

/*
 * Fused FP8 quantisation (Sec. 4.3: FP8 E4M3, scale and cast in one pass over
 * memory; the granularity here is one scale per (batch, head, token block)).
 *   amax = max |x| over the block's valid tokens x d ; amax = max(amax, 1e-12)
 *   scale = amax / 448 ; code = e4m3_rne_satfinite(x * (448 / amax))
 * x_bf16 : in,  bf16 [B,H,N,d] (strides of `shape`)
 * codes  : out, uint8 E4M3 codes, same element strides as x
 * scales : out, fp32 [B,H,nb] contiguous dequantisation scales (value = decode(code) * scale)
 * flags  : must be 0
 */
int sparkattn_quant_fp8(const sparkattn_shape_t* shape, const void* x_bf16, uint8_t* codes, float* scales,
                        uint32_t flags, void* cuda_stream);

/*
 * Quantisation and block pooling in one pass (Sec. 4.3 fuses scaling and
 * casting into a single pass over memory; here the selection's block pooling
 * rides on the same pass, so that in the FP8 configuration Q and K are read
 * from HBM once for selection and quantisation together).
 *
 * sparkattn_quant_fp8_pooled: sparkattn_quant_fp8 (same codes, same scales,
 *   bit for bit) that also writes the pooled fp32 block means of x -- steps 1
 *   and 2 of the selection rule above, same order of additions, same divide --
 *   into a selection workspace.  key_side: 0 = x is the query tensor, 1 = x is
 *   the key tensor.  select_workspace: the workspace a later
 *   sparkattn_select_pooled call takes (>= sparkattn_workspace_bytes(shape, 0,
 *   topk) bytes, 256-byte aligned); only its pooled-means region is written.
 * sparkattn_select_pooled: steps 3 to 5 of the selection rule on a workspace
 *   that one query-side and one key-side call above have filled (same shape,
 *   same stream order); outputs as sparkattn_select.  The three calls together
 *   give the same lists as sparkattn_select on the same Q and K.
 * Plain layout only (no causal window, no per-block token counts).
 */
int sparkattn_quant_fp8_pooled(const sparkattn_shape_t* shape, const void* x_bf16, uint8_t* codes, float* scales,
                               int32_t key_side, void* select_workspace, size_t workspace_bytes, void* cuda_stream);
int sparkattn_select_pooled(const sparkattn_shape_t* shape, int32_t topk, int32_t* kept_idx, int32_t* kept_cnt,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Per-token FP8 quantisation: the activation-quantisation kernel at the
 * paper's own granularity (Sec. 4.3: one dynamic scale per token row, scale
 * and cast in one pass).  Same arithmetic as sparkattn_quant_fp8 with the token
 * block replaced by one token row: amax over the row's d channels, clamped at
 * 1e-12; scale = amax / 448; code = e4m3_rne_satfinite(x * (448 / amax)).
 * Not consumed by sparkattn_fwd (which takes per-block scales); provided for
 * the activation path around it.  `shape->block` is ignored beyond validation.
 * x_bf16 : in,  bf16 [B,H,N,d] (strides of `shape`)
 * codes  : out, uint8 E4M3 codes, same element strides as x
 * scales : out, fp32 [B,H,N] contiguous
 */
int sparkattn_quant_fp8_per_token(const sparkattn_shape_t* shape, const void* x_bf16, uint8_t* codes,
                                  float* scales, void* cuda_stream);

/*
 * Block-sparse attention forward (Sec. 2 dense attention formula restricted
 * to the kept tiles; Sec. 4.1 sparse branch).  For query token i in query
 * block qb, over the keys j of the kept key blocks kept_idx[b,h,qb,0..cnt):
 *   out[i,:] = sum_j softmax_j(scale * q_i . k_j) v_j ,  lse[i] = ln sum_j exp(scale * q_i . k_j)
 * Keys >= N in a ragged last block are masked.  cnt = 0 gives out = 0, lse = -inf.
 *
 * dtype      : SPARKATTN_BF16: q,k,v bf16.  SPARKATTN_FP8_E4M3: q,k,v are E4M3
 *              codes from sparkattn_quant_fp8 with q_scale/k_scale/v_scale fp32
 *              [B,H,nb]; requires d = 128 (block 64 or 128).  Scales are NULL for bf16.
 * kept_idx   : in, int32 [B,H,nb,kmax]; entries distinct, each in [0, nb); kmax <= 2048
 *              (longer lists return SPARKATTN_E_UNSUPPORTED_SHAPE)
 * kept_cnt   : in, int32 [B,H,nb] with 0 <= cnt <= kmax; NULL means cnt = kmax everywhere
 * out_bf16   : out, bf16 [B,H,N,d], same strides as q
 * lse        : out, fp32 [B,H,N] contiguous (natural log); may be NULL
 * workspace  : >= sparkattn_workspace_bytes(shape, 1, kmax) bytes, 256-byte aligned
 * Accumulation, row maximum and row sum are fp32; P is rounded to the input
 * dtype for the second product.  The kept blocks of a list may come in any
 * order and are processed in an order of the library's choosing (the query
 * block's own key block first); the same inputs always give the same bits.
 * Out-of-range entries of a list are skipped and reported through the status
 * word of the workspace (SPARKATTN_E_BAD_INDEX).
 */
int sparkattn_fwd(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
                  const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                  const int32_t* kept_cnt, int32_t kmax, void* out_bf16, float* lse, void* workspace,
                  size_t workspace_bytes, void* cuda_stream);

/*
 * Causal frame window (Sec. 1, the auto-regressive extension: the paper says
 * the attention may be limited to a causal window and gives no formula, so
 * the reading is:)  tokens come in frames of
 * `frame_tokens` consecutive tokens; key token j counts for query token i iff
 *     i / frame_tokens - window_frames  <  j / frame_tokens  <=  i / frame_tokens.
 * sparkattn_select_window ranks only the key blocks that hold such a key for
 * some row of the query block (a contiguous run of blocks): kept_cnt =
 * min(topk, candidates) (kept_cnt must not be NULL) and the unused tail of a
 * list is -1.  sparkattn_fwd_window evaluates the same softmax attention as
 * sparkattn_fwd over the kept blocks with the token-exact window mask; a query
 * row without any admissible kept key gives a zero output row and lse = -inf.
 * All other arguments, layouts and errors are those of sparkattn_select /
 * sparkattn_fwd; frame_tokens < 1 or window_frames < 1 is SPARKATTN_E_INVALID_ARG.
 */
int sparkattn_select_window(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                            int32_t frame_tokens, int32_t window_frames, int32_t* kept_idx, int32_t* kept_cnt,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
int sparkattn_fwd_window(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
                         const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                         const int32_t* kept_cnt, int32_t kmax, int32_t frame_tokens, int32_t window_frames,
                         void* out_bf16, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Tokens stored brick by brick.  The paper partitions the sequence into
 * contiguous blocks (Sec. 2) and does not fix the order of the tokens; with
 * the raster order n = (t*Hg + y)*Wg + x a block is a strip of grid rows.
 * Here the (T, Hg, Wg) grid is cut into bricks of bt x bh x bw cells with
 * bt*bh*bw <= block (bricks at the far faces are cut to what the grid holds),
 * the bricks follow one another in raster order of the brick grid, the cells
 * of a brick in raster order inside it, and every brick takes one whole block
 * of the reordered tensors: its cells first, zero padding rows after them.
 * A block is then a compact box of the video; the reordered tensors have
 * N' = bricks * block tokens, and block_valid[b] says how many rows of block
 * b are real.  Padding rows are not keys, do not enter the pooled means of
 * the selection, and their output rows are to be ignored.
 *
 * sparkattn_brick_count : bricks of the layout (host arithmetic; 0 for invalid
 *                         arguments): the nb of the reordered tensors
 * sparkattn_brick_layout: grid_host, brick_host HOST int32[3]; block 64 or 128.
 *     gather_index  out, device int32 [bricks*block]: raster index of the token
 *                   at each padded position, -1 for padding (gather raster ->
 *                   bricks); may be NULL
 *     block_valid   out, device int32 [bricks]; may be NULL
 *     scatter_index out, device int32 [N]: padded position of raster token n
 *                   (gather bricks -> raster); may be NULL (not all three)
 * sparkattn_gather_tokens: out[b,h,i,:] = x[b,h,index[i],:] for i < N of
 *     dst_shape, one pass over memory; x bf16 with src_shape, out bf16 with
 *     dst_shape (same B, H, d; the two must not overlap); index device int32
 *     [dst N]: -1 leaves a zero row, any other value outside [0, src N) leaves
 *     a zero row and sets SPARKATTN_E_BAD_INDEX in the status word of
 *     `workspace` (>= sparkattn_workspace_bytes(shape, 2, 0) = 256 bytes,
 *     256-byte aligned; only the status header is used).
 * sparkattn_select_padded / sparkattn_fwd_padded: sparkattn_select /
 *     sparkattn_fwd on reordered tensors (N a multiple of the block size;
 *     d = 128 with 128- or 64-token blocks, else SPARKATTN_E_UNSUPPORTED_SHAPE) with
 *     block_valid device int32 [nb], every entry in [1, block]: pooled means
 *     over the real rows of a block, keys beyond block_valid[kb] of a kept
 *     block get weight 0.  Output rows of padding queries hold finite values
 *     without meaning.  All other arguments as in the plain calls.
 */
int64_t sparkattn_brick_count(const int32_t* grid_host, const int32_t* brick_host);
int sparkattn_brick_layout(const int32_t* grid_host, const int32_t* brick_host, int32_t block, int32_t* gather_index,
                           int32_t* block_valid, int32_t* scatter_index, void* cuda_stream);
int sparkattn_gather_tokens(const sparkattn_shape_t* src_shape, const void* x_bf16, const sparkattn_shape_t* dst_shape,
                            const int32_t* index, void* out_bf16, void* workspace, size_t workspace_bytes,
                            void* cuda_stream);
int sparkattn_select_padded(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                            const int32_t* block_valid, int32_t* kept_idx, int32_t* kept_cnt, void* workspace,
                            size_t workspace_bytes, void* cuda_stream);
int sparkattn_fwd_padded(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
                         const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                         const int32_t* kept_cnt, int32_t kmax, const int32_t* block_valid, void* out_bf16, float* lse,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Synchronises the stream and returns the device status word of a workspace
 * (SPARKATTN_OK, SPARKATTN_E_BAD_INDEX or SPARKATTN_E_DEVICE_TIMEOUT). */
int sparkattn_read_status(void* workspace, void* cuda_stream);

/*
 * Whole path on HOST buffers: copies Q, K, V to the device arena, runs
 * select (+ quant for FP8) + fwd, copies the output back and synchronises.
 * q_host, k_host, v_host, out_host: contiguous bf16 [B,H,N,d] in (preferably
 * pinned) host memory; kept_idx_host may be NULL or int32 [B,H,nb,topk] to
 * receive the selected lists.  arena: device scratch of at least
 * sparkattn_arena_bytes(shape, dtype, topk) bytes, 256-byte aligned.
 * The heads are independent, so the call runs as a pipeline over groups of
 * heads (about eight groups, at most 16; a group never spans two batch
 * entries, so B > 16 returns SPARKATTN_E_UNSUPPORTED_SHAPE): while one group is selected and
 * attended on `cuda_stream`, the next is copied in and the previous one's
 * output copied out on two copy streams that the library creates once per
 * device and keeps; both are ordered after work already queued on
 * `cuda_stream`, and `cuda_stream` ends after the last copy.  With pageable
 * host memory the copies are staged by the driver and the overlap is lost;
 * the result is the same.  Returns the first non-zero device status of any
 * group (SPARKATTN_E_BAD_INDEX, SPARKATTN_E_DEVICE_TIMEOUT), an argument or
 * CUDA error, or SPARKATTN_OK; on an error the output is undefined.
 */
size_t sparkattn_arena_bytes(const sparkattn_shape_t* shape, int32_t dtype, int32_t topk);
int sparkattn_attention_host(const sparkattn_shape_t* shape, int32_t dtype, const void* q_host,
                             const void* k_host, const void* v_host, int32_t topk, void* out_host,
                             int32_t* kept_idx_host, void* arena, size_t arena_bytes, void* cuda_stream);

/*
 * Low-rank compensation branch and gate fusion (Sec. 4.1, "low-rank
 * compensation branch" and the fused output O = O_s + g * r * O_lr).
 * With rank r = 64 projections P_q, P_k per head and the rank-truncated rotary
 * rotation R_r (adjacent feature pairs (2m, 2m+1) rotated by the angle
 * pos_axis[m] * freq[m], pos = the token's (t, y, x) coordinate on the latent
 * grid, raster token order n = (t * Hg + y) * Wg + x):
 *   q~_i = R_r(p_i) silu(P_q q_i)        k~_j = R_r(p_j) silu(P_k k_j)
 *   C    = sum_j k~_j v_j^T              (r x d per (batch, head): sparkattn_comp_state)
 *   y_i  = q~_i^T C ;  O_lr,i = y_i / sqrt(mean_c y_i[c]^2 + eps)      (RMSNorm, no weight)
 *   r_i  = sqrt(mean_c O_s,i[c]^2)  ;    O_i = O_s,i + g_i * r_i * O_lr,i   (sparkattn_comp_apply)
 * Linear in N.  Requires d = 128 and rank = 64; `shape->block` is validated but not used.
 *
 * Arithmetic: projections, C and y are tensor-core products of bf16 operands
 * with fp32 accumulation (q~, k~ and, in the apply pass, C are rounded to
 * bf16 first); silu, rotation, norms and the fusion are fp32; the state is
 * summed over fixed token chunks in a fixed order.
 *
 * k, v, q, o_sparse : in,  bf16 [B,H,N,d] with the strides of `shape`
 * pk, pq            : in,  bf16 [H, rank, d] contiguous, 16-byte aligned
 * grid_host         : in,  HOST int32[3] = (T, Hg, Wg), T*Hg*Wg = N
 * rope_axis_host    : in,  HOST int32[rank/2], entries 0 (t), 1 (y) or 2 (x)
 * rope_freq_host    : in,  HOST fp32[rank/2]
 * state             : comp_state out / comp_apply in, fp32 [B,H,rank,d] contiguous
 * gate              : in,  fp32 [B,H,N] contiguous (the token-wise gate g)
 * out_bf16          : out, bf16 [B,H,N,d], strides of `shape`; may alias o_sparse
 * eps               : RMSNorm epsilon (> 0)
 * workspace         : >= sparkattn_comp_workspace_bytes(shape, grid_host) bytes, 256-byte aligned
 *                     (sized for the state pass; the apply pass needs only its first
 *                     512 + 4 * rank * (T + Hg + Wg) bytes); first word = device status
 * The host arrays are read during the call only.
 */
size_t sparkattn_comp_workspace_bytes(const sparkattn_shape_t* shape, const int32_t* grid_host);
int sparkattn_comp_state(const sparkattn_shape_t* shape, const void* k_bf16, const void* v_bf16, const void* pk_bf16,
                         int32_t rank, const int32_t* grid_host, const int32_t* rope_axis_host,
                         const float* rope_freq_host, float* state, void* workspace, size_t workspace_bytes,
                         void* cuda_stream);
int sparkattn_comp_apply(const sparkattn_shape_t* shape, const void* q_bf16, const void* pq_bf16, int32_t rank,
                         const int32_t* grid_host, const int32_t* rope_axis_host, const float* rope_freq_host,
                         const float* state, const float* gate, const void* o_sparse_bf16, void* out_bf16, float eps,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Sparse forward and gate fusion in one kernel (Sec. 4.1: the module's output
 * O = O_s + g * r * O_lr, with O_s the block-sparse attention output).
 *
 * Equivalent to sparkattn_fwd (bf16) followed by sparkattn_comp_apply with
 * o_sparse = that call's output, without the round trip of O_s and the second
 * read of Q through device memory: the warpgroup that finishes a query block
 * keeps the normalised, bf16-rounded O_s rows in registers, forms
 * q~ = R_r(p) silu(P_q q) from the Q tile still in shared memory, y = q~^T C
 * on the tensor cores, and writes O_s + g * r * y / rms(y).  Every step is
 * taken in the arithmetic and order of the two separate calls, so the output
 * equals theirs bit for bit.  The state C comes from sparkattn_comp_state.
 *
 * Requires bf16 operands, d = 128, block = 128, rank = 64; no window mask and
 * no padded-brick layout (SPARKATTN_E_UNSUPPORTED_SHAPE otherwise).
 *
 * q, k, v           : in,  bf16 [B,H,N,d] with the strides of `shape`
 * kept_idx, kept_cnt, kmax, lse : as in sparkattn_fwd (lse is that of O_s)
 * pq, grid_host, rope_axis_host, rope_freq_host, state, gate, eps : as in sparkattn_comp_apply
 * out_bf16          : out, bf16 [B,H,N,d], strides of `shape`
 * workspace         : >= sparkattn_fwd_gated_workspace_bytes(shape, kmax, grid_host) bytes
 *                     (0 = unsupported arguments), 256-byte aligned; first word = device status
 * Errors as in sparkattn_fwd and sparkattn_comp_apply; on an error the output is undefined.
 */
size_t sparkattn_fwd_gated_workspace_bytes(const sparkattn_shape_t* shape, int32_t kmax, const int32_t* grid_host);
int sparkattn_fwd_gated(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, const void* v_bf16,
                        const int32_t* kept_idx, const int32_t* kept_cnt, int32_t kmax, const void* pq_bf16,
                        int32_t rank, const int32_t* grid_host, const int32_t* rope_axis_host,
                        const float* rope_freq_host, const float* state, const float* gate, float eps, void* out_bf16,
                        float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Block selection without any allocation (the paper has no counterpart: this
 * is a packaging variant of sparkattn_select, same rule, same outputs).
 *
 * For callers that may not allocate device memory when they call: a serving
 * loop whose memory budget was fixed at start-up, a host application whose
 * allocator is frozen after initialisation, a plugin that only receives its
 * input and output buffers.  The scratch that sparkattn_select takes as a
 * workspace lives here in a fixed device array inside the library image, of
 * sparkattn_select_noalloc_max_bytes() bytes (32 MiB), which every GPU that
 * loads the library holds until the process exits.  The call itself performs
 * no cudaMalloc / cudaFree and calls no allocating library routine.
 *
 *   - Arguments as for sparkattn_select, minus the workspace.  q_bf16, k_bf16,
 *     kept_idx, kept_cnt are caller-owned device buffers.
 *   - A shape whose scratch need (sparkattn_workspace_bytes(shape, 0, topk))
 *     exceeds the array returns SPARKATTN_E_WORKSPACE_TOO_SMALL and enqueues
 *     nothing; the other argument errors are those of sparkattn_select.
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and caches it; make that first call before starting
 *     any stream capture.
 *   - All calls on a device share the one array, which still holds the previous
 *     call's contents; the library clears what must start at zero.  Calls whose
 *     kernels can overlap on the GPU (different streams or threads) race on it:
 *     serialise them.
 *   - sparkattn_select_noalloc_status synchronises the stream and returns the
 *     device status word of the last call on the current device.
 */
size_t sparkattn_select_noalloc_max_bytes(void);
int sparkattn_select_noalloc(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                             int32_t* kept_idx, int32_t* kept_cnt, void* cuda_stream);
int sparkattn_select_noalloc_status(void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPARKATTN_H_ */
