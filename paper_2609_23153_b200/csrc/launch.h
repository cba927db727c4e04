// Internal host-side launch interface between the C-ABI layer (api.cu) and the
// kernel translation units.  Every launcher validates nothing: api.cu has
// already checked the arguments.  Each returns a sparkattn_status.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sparkattn.h"

namespace sparkattn {

// quant.cu
int launch_quant_fp8(const sparkattn_shape_t& s, const void* x, uint8_t* codes, float* scales,
                     cudaStream_t stream);

// quantisation + the selection's pooled block means in one pass (pooled: see select_pooled_ptr)
int launch_quant_fp8_pooled(const sparkattn_shape_t& s, const void* x, uint8_t* codes, float* scales, float* pooled,
                            bool key_side, cudaStream_t stream);

int launch_quant_fp8_per_token(const sparkattn_shape_t& s, const void* x, uint8_t* codes, float* scales,
                               cudaStream_t stream);

// select.cu
constexpr int kSelectMaxBlocks = 4096;  // largest nb the selection kernel holds in shared memory
size_t select_workspace_bytes(const sparkattn_shape_t& s);
// frame_tokens = 0: no causal window; otherwise window >= 1 frames of frame_tokens tokens
// block_valid: real tokens per block when bricks are padded to whole blocks (device int32 [nb]), else NULL
int launch_select(const sparkattn_shape_t& s, const void* q, const void* k, int topk, int frame_tokens, int window,
                  const int32_t* block_valid, int32_t* kept_idx, int32_t* kept_cnt, void* workspace, cudaStream_t stream);

// pooled means inside a selection workspace (query side / key side), and scores + top-k on means already there
float* select_pooled_ptr(const sparkattn_shape_t& s, void* workspace, bool key_side);
int launch_select_pooled(const sparkattn_shape_t& s, int topk, int32_t* kept_idx, int32_t* kept_cnt, void* workspace,
                         cudaStream_t stream);

// fwd.cu
constexpr int kFwdMaxKept = 2048;  // longest kept list (kmax) the forward kernel stages in shared memory
size_t fwd_workspace_bytes(const sparkattn_shape_t& s, int kmax);
int launch_fwd(const sparkattn_shape_t& s, int dtype, const void* q, const void* k, const void* v,
               const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
               const int32_t* kept_cnt, int kmax, int frame_tokens, int window, const int32_t* block_valid, void* out,
               float* lse, void* workspace, cudaStream_t stream);

// fwd_pipe.cu: persistent pipelined forward for d = 128, block = 128 (bf16 and FP8)
bool fwd_pipe_supported(const sparkattn_shape_t& s);   // d = 128 with 128-token blocks, or 64-token blocks (paired)
size_t fwd_pipe_workspace_bytes(const sparkattn_shape_t& s, int kmax);
int launch_fwd_pipe(const sparkattn_shape_t& s, bool fp8, const void* q, const void* k, const void* v,
                    const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                    const int32_t* kept_cnt, int kmax, int frame_tokens, int window, const int32_t* block_valid,
                    void* out, float* lse, void* workspace, cudaStream_t stream);

// comp.cu
constexpr int kCompRank = 64;  // rank of the compensation branch the kernels are built for
// header + rotary table (+ the per-chunk partial states of the state pass)
size_t comp_workspace_bytes(const sparkattn_shape_t& s, const int32_t* grid, bool with_state);
int launch_comp_state(const sparkattn_shape_t& s, const void* k, const void* v, const void* pk, const int32_t* grid,
                      const int32_t* axis, const float* freq, float* state, void* workspace, cudaStream_t stream);
int launch_comp_apply(const sparkattn_shape_t& s, const void* q, const void* pq, const int32_t* grid,
                      const int32_t* axis, const float* freq, const float* state, const float* gate,
                      const void* o_sparse, void* out, float eps, void* workspace, cudaStream_t stream);

// fwd_pipe.cu: forward whose epilogue adds the gated compensation term (bf16, d = 128, 128-token blocks);
// workspace = that of the plain forward, rounded up to 256 bytes, then the rotary table
bool fwd_pipe_gated_supported(const sparkattn_shape_t& s);
size_t fwd_pipe_gated_workspace_bytes(const sparkattn_shape_t& s, int kmax, const int32_t* grid);
int launch_fwd_pipe_gated(const sparkattn_shape_t& s, const void* q, const void* k, const void* v,
                          const int32_t* kept_idx, const int32_t* kept_cnt, int kmax, const void* pq,
                          const int32_t* grid, const int32_t* axis, const float* freq, const float* state,
                          const float* gate, float eps, void* out, float* lse, void* workspace, cudaStream_t stream);

// reorder.cu: tokens stored brick by brick, every brick padded to a whole block
int launch_brick_layout(const int32_t* grid, const int32_t* brick, int block, int32_t* gather, int32_t* block_valid,
                        int32_t* scatter, cudaStream_t stream);
int launch_gather_tokens(const sparkattn_shape_t& src, const void* x, const sparkattn_shape_t& dst, const int32_t* index,
                         void* out, void* workspace, cudaStream_t stream);

}  // namespace sparkattn
