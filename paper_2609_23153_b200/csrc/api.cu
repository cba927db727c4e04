// C-ABI layer of sparkattn: argument validation, workspace sizing and the
// host-buffer convenience path.  All device work is in select.cu, quant.cu and
// fwd.cu; nothing here touches tensor data on the CPU.
#include <math.h>
#include <string.h>

#include <mutex>

#include "common.cuh"
#include "launch.h"

using namespace sparkattn;

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int check_shape(const sparkattn_shape_t* s) {
  if (s == nullptr) return SPARKATTN_E_INVALID_ARG;
  if (s->struct_size != sizeof(sparkattn_shape_t) || s->version != SPARKATTN_VERSION) return SPARKATTN_E_INVALID_ARG;
  if (s->B < 1 || s->H < 1 || s->N < 1 || s->reserved != 0 || s->pad != 0) return SPARKATTN_E_INVALID_ARG;
  if (!(s->softmax_scale >= 0.0f) || isinf(s->softmax_scale)) return SPARKATTN_E_INVALID_ARG;
  if (!((s->d == 64 && s->block == 64) || (s->d == 128 && (s->block == 128 || s->block == 64))))
    return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (s->stride_n < s->d || s->stride_h < 1 || s->stride_b < 1) return SPARKATTN_E_INVALID_ARG;
  // 16-byte rule for vector loads and TMA, for 2-byte and for 1-byte elements
  if (s->stride_n % 16 || s->stride_h % 16 || s->stride_b % 16) return SPARKATTN_E_MISALIGNED;
  if ((long long)s->B * s->H > 65535LL * 32768LL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  return SPARKATTN_OK;
}

inline int num_blocks(const sparkattn_shape_t* s) { return (s->N + s->block - 1) / s->block; }

}  // namespace

extern "C" {

int sparkattn_version(void) { return SPARKATTN_VERSION; }

const char* sparkattn_status_string(int status) {
  switch (status) {
    case SPARKATTN_OK: return "ok";
    case SPARKATTN_E_INVALID_ARG: return "invalid argument";
    case SPARKATTN_E_UNSUPPORTED_SHAPE: return "unsupported shape";
    case SPARKATTN_E_MISALIGNED: return "misaligned pointer or stride";
    case SPARKATTN_E_WORKSPACE_TOO_SMALL: return "workspace too small";
    case SPARKATTN_E_CUDA: return "CUDA error";
    case SPARKATTN_E_DEVICE_TIMEOUT: return "device-side wait timed out";
    case SPARKATTN_E_BAD_INDEX: return "kept block index out of range";
    case SPARKATTN_E_NO_DEVICE: return "no CUDA device or driver entry point";
    default: return "unknown status";
  }
}

size_t sparkattn_workspace_bytes(const sparkattn_shape_t* shape, int32_t which, int32_t topk_or_kmax) {
  if (check_shape(shape) != SPARKATTN_OK) return 0;
  if (which == 0) return select_workspace_bytes(*shape);
  if (which == 1) return topk_or_kmax >= 1 ? fwd_workspace_bytes(*shape, topk_or_kmax) : 0;
  if (which == 2) return kWorkspaceHeaderBytes;   // sparkattn_gather_tokens: the status header only
  return 0;
}

namespace {
int select_impl(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                int32_t frame_tokens, int32_t window, const int32_t* block_valid, int32_t* kept_idx, int32_t* kept_cnt,
                void* workspace, size_t workspace_bytes, void* cuda_stream);
}  // namespace

int sparkattn_select(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                     int32_t* kept_idx, int32_t* kept_cnt, void* workspace, size_t workspace_bytes,
                     void* cuda_stream) {
  return select_impl(shape, q_bf16, k_bf16, topk, 0, 0, nullptr, kept_idx, kept_cnt, workspace, workspace_bytes,
                     cuda_stream);
}

int sparkattn_select_window(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                            int32_t frame_tokens, int32_t window_frames, int32_t* kept_idx, int32_t* kept_cnt,
                            void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (frame_tokens < 1 || window_frames < 1 || kept_cnt == nullptr) return SPARKATTN_E_INVALID_ARG;
  return select_impl(shape, q_bf16, k_bf16, topk, frame_tokens, window_frames, nullptr, kept_idx, kept_cnt, workspace,
                     workspace_bytes, cuda_stream);
}

namespace {
int select_impl(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                int32_t frame_tokens, int32_t window, const int32_t* block_valid, int32_t* kept_idx, int32_t* kept_cnt,
                void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (!q_bf16 || !k_bf16 || !kept_idx || !workspace) return SPARKATTN_E_INVALID_ARG;
  const int nb = num_blocks(shape);
  if (topk < 1 || topk > nb) return SPARKATTN_E_INVALID_ARG;
  if (nb > kSelectMaxBlocks) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (!aligned16(q_bf16) || !aligned16(k_bf16) || !aligned256(workspace)) return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < select_workspace_bytes(*shape)) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  return launch_select(*shape, q_bf16, k_bf16, topk, frame_tokens, window, block_valid, kept_idx, kept_cnt, workspace,
                       stream);
}
}  // namespace

int sparkattn_quant_fp8(const sparkattn_shape_t* shape, const void* x_bf16, uint8_t* codes, float* scales,
                        uint32_t flags, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (!x_bf16 || !codes || !scales || flags != 0) return SPARKATTN_E_INVALID_ARG;
  if (!aligned16(x_bf16) || !aligned16(codes)) return SPARKATTN_E_MISALIGNED;
  return launch_quant_fp8(*shape, x_bf16, codes, scales, static_cast<cudaStream_t>(cuda_stream));
}

int sparkattn_quant_fp8_pooled(const sparkattn_shape_t* shape, const void* x_bf16, uint8_t* codes, float* scales,
                               int32_t key_side, void* select_workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (!x_bf16 || !codes || !scales || !select_workspace || (key_side != 0 && key_side != 1)) return SPARKATTN_E_INVALID_ARG;
  if (num_blocks(shape) > kSelectMaxBlocks) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (!aligned16(x_bf16) || !aligned16(codes) || !aligned256(select_workspace)) return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < select_workspace_bytes(*shape)) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  return launch_quant_fp8_pooled(*shape, x_bf16, codes, scales, select_pooled_ptr(*shape, select_workspace, key_side != 0),
                                 key_side != 0, static_cast<cudaStream_t>(cuda_stream));
}

int sparkattn_select_pooled(const sparkattn_shape_t* shape, int32_t topk, int32_t* kept_idx, int32_t* kept_cnt,
                            void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (!kept_idx || !workspace) return SPARKATTN_E_INVALID_ARG;
  const int nb = num_blocks(shape);
  if (topk < 1 || topk > nb) return SPARKATTN_E_INVALID_ARG;
  if (nb > kSelectMaxBlocks) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (!aligned256(workspace)) return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < select_workspace_bytes(*shape)) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  return launch_select_pooled(*shape, topk, kept_idx, kept_cnt, workspace, stream);
}

int sparkattn_quant_fp8_per_token(const sparkattn_shape_t* shape, const void* x_bf16, uint8_t* codes,
                                  float* scales, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (!x_bf16 || !codes || !scales) return SPARKATTN_E_INVALID_ARG;
  if (!aligned16(x_bf16) || !aligned16(codes)) return SPARKATTN_E_MISALIGNED;
  return launch_quant_fp8_per_token(*shape, x_bf16, codes, scales, static_cast<cudaStream_t>(cuda_stream));
}

namespace {
int fwd_impl(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
             const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
             const int32_t* kept_cnt, int32_t kmax, int32_t frame_tokens, int32_t window, const int32_t* block_valid,
             void* out_bf16, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream);
}  // namespace

int sparkattn_fwd(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
                  const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                  const int32_t* kept_cnt, int32_t kmax, void* out_bf16, float* lse, void* workspace,
                  size_t workspace_bytes, void* cuda_stream) {
  return fwd_impl(shape, dtype, q, k, v, q_scale, k_scale, v_scale, kept_idx, kept_cnt, kmax, 0, 0, nullptr, out_bf16, lse,
                  workspace, workspace_bytes, cuda_stream);
}

int sparkattn_fwd_window(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
                         const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                         const int32_t* kept_cnt, int32_t kmax, int32_t frame_tokens, int32_t window_frames,
                         void* out_bf16, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (frame_tokens < 1 || window_frames < 1) return SPARKATTN_E_INVALID_ARG;
  return fwd_impl(shape, dtype, q, k, v, q_scale, k_scale, v_scale, kept_idx, kept_cnt, kmax, frame_tokens,
                  window_frames, nullptr, out_bf16, lse, workspace, workspace_bytes, cuda_stream);
}

namespace {
int fwd_impl(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
             const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
             const int32_t* kept_cnt, int32_t kmax, int32_t frame_tokens, int32_t window, const int32_t* block_valid,
             void* out_bf16, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (dtype != SPARKATTN_BF16 && dtype != SPARKATTN_FP8_E4M3) return SPARKATTN_E_INVALID_ARG;
  if (!q || !k || !v || !kept_idx || !out_bf16 || !workspace) return SPARKATTN_E_INVALID_ARG;
  if (kmax < 1 || kmax > num_blocks(shape)) return SPARKATTN_E_INVALID_ARG;
  if (kmax > kFwdMaxKept) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (dtype == SPARKATTN_FP8_E4M3) {
    if (!q_scale || !k_scale || !v_scale) return SPARKATTN_E_INVALID_ARG;
    if (shape->d != 128) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  }
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out_bf16) || !aligned256(workspace))
    return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < fwd_workspace_bytes(*shape, kmax)) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  return launch_fwd(*shape, dtype, q, k, v, q_scale, k_scale, v_scale, kept_idx, kept_cnt, kmax, frame_tokens, window,
                    block_valid, out_bf16, lse, workspace, static_cast<cudaStream_t>(cuda_stream));
}
}  // namespace

namespace {
int check_comp(const sparkattn_shape_t* s, int32_t rank, const int32_t* grid, const int32_t* axis, const float* freq) {
  int rc = check_shape(s);
  if (rc != SPARKATTN_OK) return rc;
  if (!grid || !axis || !freq) return SPARKATTN_E_INVALID_ARG;
  if (s->d != 128 || rank != kCompRank) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (grid[0] < 1 || grid[1] < 1 || grid[2] < 1 || (long long)grid[0] * grid[1] * grid[2] != (long long)s->N)
    return SPARKATTN_E_INVALID_ARG;
  for (int m = 0; m < rank / 2; ++m)
    if (axis[m] < 0 || axis[m] > 2 || !isfinite(freq[m])) return SPARKATTN_E_INVALID_ARG;
  return SPARKATTN_OK;
}
}  // namespace

size_t sparkattn_comp_workspace_bytes(const sparkattn_shape_t* shape, const int32_t* grid_host) {
  if (check_shape(shape) != SPARKATTN_OK || shape->d != 128 || !grid_host) return 0;
  if (grid_host[0] < 1 || grid_host[1] < 1 || grid_host[2] < 1 ||
      (long long)grid_host[0] * grid_host[1] * grid_host[2] != (long long)shape->N)
    return 0;
  return comp_workspace_bytes(*shape, grid_host, true);
}

int sparkattn_comp_state(const sparkattn_shape_t* shape, const void* k_bf16, const void* v_bf16, const void* pk_bf16,
                         int32_t rank, const int32_t* grid_host, const int32_t* rope_axis_host,
                         const float* rope_freq_host, float* state, void* workspace, size_t workspace_bytes,
                         void* cuda_stream) {
  int rc = check_comp(shape, rank, grid_host, rope_axis_host, rope_freq_host);
  if (rc != SPARKATTN_OK) return rc;
  if (!k_bf16 || !v_bf16 || !pk_bf16 || !state || !workspace) return SPARKATTN_E_INVALID_ARG;
  if (!aligned16(k_bf16) || !aligned16(v_bf16) || !aligned16(pk_bf16) || !aligned16(state) || !aligned256(workspace))
    return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < comp_workspace_bytes(*shape, grid_host, true)) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  return launch_comp_state(*shape, k_bf16, v_bf16, pk_bf16, grid_host, rope_axis_host, rope_freq_host, state,
                           workspace, static_cast<cudaStream_t>(cuda_stream));
}

int sparkattn_comp_apply(const sparkattn_shape_t* shape, const void* q_bf16, const void* pq_bf16, int32_t rank,
                         const int32_t* grid_host, const int32_t* rope_axis_host, const float* rope_freq_host,
                         const float* state, const float* gate, const void* o_sparse_bf16, void* out_bf16, float eps,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check_comp(shape, rank, grid_host, rope_axis_host, rope_freq_host);
  if (rc != SPARKATTN_OK) return rc;
  if (!q_bf16 || !pq_bf16 || !state || !gate || !o_sparse_bf16 || !out_bf16 || !workspace)
    return SPARKATTN_E_INVALID_ARG;
  if (!(eps > 0.0f) || isinf(eps)) return SPARKATTN_E_INVALID_ARG;
  if (!aligned16(q_bf16) || !aligned16(pq_bf16) || !aligned16(state) || !aligned16(o_sparse_bf16) ||
      !aligned16(out_bf16) || !aligned256(workspace))
    return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < comp_workspace_bytes(*shape, grid_host, false)) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  return launch_comp_apply(*shape, q_bf16, pq_bf16, grid_host, rope_axis_host, rope_freq_host, state, gate,
                           o_sparse_bf16, out_bf16, eps, workspace, static_cast<cudaStream_t>(cuda_stream));
}

size_t sparkattn_fwd_gated_workspace_bytes(const sparkattn_shape_t* shape, int32_t kmax, const int32_t* grid_host) {
  if (check_shape(shape) != SPARKATTN_OK || !fwd_pipe_gated_supported(*shape) || !grid_host) return 0;
  if (kmax < 1 || kmax > num_blocks(shape) || kmax > kFwdMaxKept) return 0;
  if (grid_host[0] < 1 || grid_host[1] < 1 || grid_host[2] < 1 ||
      (long long)grid_host[0] * grid_host[1] * grid_host[2] != (long long)shape->N)
    return 0;
  return fwd_pipe_gated_workspace_bytes(*shape, kmax, grid_host);
}

int sparkattn_fwd_gated(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, const void* v_bf16,
                        const int32_t* kept_idx, const int32_t* kept_cnt, int32_t kmax, const void* pq_bf16,
                        int32_t rank, const int32_t* grid_host, const int32_t* rope_axis_host,
                        const float* rope_freq_host, const float* state, const float* gate, float eps, void* out_bf16,
                        float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = check_comp(shape, rank, grid_host, rope_axis_host, rope_freq_host);
  if (rc != SPARKATTN_OK) return rc;
  if (!fwd_pipe_gated_supported(*shape)) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (!q_bf16 || !k_bf16 || !v_bf16 || !kept_idx || !pq_bf16 || !state || !gate || !out_bf16 || !workspace)
    return SPARKATTN_E_INVALID_ARG;
  if (kmax < 1 || kmax > num_blocks(shape)) return SPARKATTN_E_INVALID_ARG;
  if (kmax > kFwdMaxKept) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  if (!(eps > 0.0f) || isinf(eps)) return SPARKATTN_E_INVALID_ARG;
  if (!aligned16(q_bf16) || !aligned16(k_bf16) || !aligned16(v_bf16) || !aligned16(pq_bf16) || !aligned16(state) ||
      !aligned16(out_bf16) || !aligned256(workspace))
    return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < fwd_pipe_gated_workspace_bytes(*shape, kmax, grid_host)) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  return launch_fwd_pipe_gated(*shape, q_bf16, k_bf16, v_bf16, kept_idx, kept_cnt, kmax, pq_bf16, grid_host,
                               rope_axis_host, rope_freq_host, state, gate, eps, out_bf16, lse, workspace,
                               static_cast<cudaStream_t>(cuda_stream));
}

namespace {
// bricks padded to whole blocks: every block is whole, so N is a multiple of the block size
int check_padded(const sparkattn_shape_t* shape, const int32_t* block_valid) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (block_valid == nullptr) return SPARKATTN_E_INVALID_ARG;
  if (shape->N % shape->block != 0) return SPARKATTN_E_INVALID_ARG;
  if (shape->d != 128) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  return SPARKATTN_OK;
}
}  // namespace

int64_t sparkattn_brick_count(const int32_t* grid_host, const int32_t* brick_host) {
  if (!grid_host || !brick_host) return 0;
  int64_t n = 1;
  for (int a = 0; a < 3; ++a) {
    if (grid_host[a] < 1 || brick_host[a] < 1) return 0;
    n *= (grid_host[a] + brick_host[a] - 1) / brick_host[a];
  }
  return n;
}

int sparkattn_brick_layout(const int32_t* grid_host, const int32_t* brick_host, int32_t block, int32_t* gather_index,
                           int32_t* block_valid, int32_t* scatter_index, void* cuda_stream) {
  const int64_t bricks = sparkattn_brick_count(grid_host, brick_host);
  if (bricks == 0 || (block != 64 && block != 128) || (!gather_index && !block_valid && !scatter_index))
    return SPARKATTN_E_INVALID_ARG;
  if ((int64_t)brick_host[0] * brick_host[1] * brick_host[2] > block) return SPARKATTN_E_INVALID_ARG;
  const int64_t n = (int64_t)grid_host[0] * grid_host[1] * grid_host[2];
  if (n > 0x7fffffffLL || bricks * block > 0x7fffffffLL) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  return launch_brick_layout(grid_host, brick_host, block, gather_index, block_valid, scatter_index,
                             static_cast<cudaStream_t>(cuda_stream));
}

int sparkattn_gather_tokens(const sparkattn_shape_t* src_shape, const void* x_bf16, const sparkattn_shape_t* dst_shape,
                            const int32_t* index, void* out_bf16, void* workspace, size_t workspace_bytes,
                            void* cuda_stream) {
  int rc = check_shape(src_shape);
  if (rc != SPARKATTN_OK) return rc;
  if ((rc = check_shape(dst_shape)) != SPARKATTN_OK) return rc;
  if (src_shape->B != dst_shape->B || src_shape->H != dst_shape->H || src_shape->d != dst_shape->d)
    return SPARKATTN_E_INVALID_ARG;
  if (!x_bf16 || !index || !out_bf16 || !workspace || x_bf16 == out_bf16) return SPARKATTN_E_INVALID_ARG;
  if (!aligned16(x_bf16) || !aligned16(out_bf16) || !aligned256(workspace)) return SPARKATTN_E_MISALIGNED;
  if (workspace_bytes < (size_t)kWorkspaceHeaderBytes) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(workspace, 0, kWorkspaceHeaderBytes, stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  return launch_gather_tokens(*src_shape, x_bf16, *dst_shape, index, out_bf16, workspace, stream);
}

int sparkattn_select_padded(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                            const int32_t* block_valid, int32_t* kept_idx, int32_t* kept_cnt, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
  const int rc = check_padded(shape, block_valid);
  if (rc != SPARKATTN_OK) return rc;
  return select_impl(shape, q_bf16, k_bf16, topk, 0, 0, block_valid, kept_idx, kept_cnt, workspace, workspace_bytes,
                     cuda_stream);
}

int sparkattn_fwd_padded(const sparkattn_shape_t* shape, int32_t dtype, const void* q, const void* k, const void* v,
                         const float* q_scale, const float* k_scale, const float* v_scale, const int32_t* kept_idx,
                         const int32_t* kept_cnt, int32_t kmax, const int32_t* block_valid, void* out_bf16, float* lse,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  const int rc = check_padded(shape, block_valid);
  if (rc != SPARKATTN_OK) return rc;
  return fwd_impl(shape, dtype, q, k, v, q_scale, k_scale, v_scale, kept_idx, kept_cnt, kmax, 0, 0, block_valid, out_bf16,
                  lse, workspace, workspace_bytes, cuda_stream);
}

int sparkattn_read_status(void* workspace, void* cuda_stream) {
  if (!workspace) return SPARKATTN_E_INVALID_ARG;
  int32_t word = 0;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return SPARKATTN_E_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return SPARKATTN_E_CUDA;
  return word;
}

// Arena layout of the host-buffer path (every region 256-byte aligned):
//   q, k, v, out (bf16) | kept_idx | kept_cnt | select workspace | fwd workspace | status words |
//   FP8 only: q/k/v codes, q/k/v scales
namespace {
struct Arena {
  size_t q, k, v, out, idx, cnt, ws_sel, ws_fwd, status, cq, ck, cv, sq, sk, sv, total;
};
Arena plan_arena(const sparkattn_shape_t& s, int dtype, int topk) {
  Arena a;
  const size_t nb = (size_t)num_blocks(&s);
  const size_t elems = (size_t)s.B * s.H * s.N * s.d;
  const size_t bhn = (size_t)s.B * s.H * nb;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes, 256); return o; };
  a.q = take(elems * 2); a.k = take(elems * 2); a.v = take(elems * 2); a.out = take(elems * 2);
  a.idx = take(bhn * topk * 4); a.cnt = take(bhn * 4);
  sparkattn_shape_t c = s;
  c.stride_n = s.d; c.stride_h = (int64_t)s.N * s.d; c.stride_b = (int64_t)s.H * s.N * s.d;
  a.ws_sel = take(select_workspace_bytes(c));
  a.ws_fwd = take(fwd_workspace_bytes(c, topk));
  a.status = take(256);
  a.cq = a.ck = a.cv = a.sq = a.sk = a.sv = 0;
  if (dtype == SPARKATTN_FP8_E4M3) {
    a.cq = take(elems); a.ck = take(elems); a.cv = take(elems);
    a.sq = take(bhn * 4); a.sk = take(bhn * 4); a.sv = take(bhn * 4);
  }
  a.total = off;
  return a;
}
}  // namespace

size_t sparkattn_arena_bytes(const sparkattn_shape_t* shape, int32_t dtype, int32_t topk) {
  if (check_shape(shape) != SPARKATTN_OK || topk < 1 || topk > num_blocks(shape)) return 0;
  return plan_arena(*shape, dtype, topk).total;
}

namespace {
// Copy streams of the host-buffer path, one pair per device, created on first use and kept.
struct HostPathStreams {
  cudaStream_t in = nullptr, out = nullptr;
};
HostPathStreams* host_path_streams() {
  static HostPathStreams per_device[64];
  static std::mutex lock;
  std::lock_guard<std::mutex> guard(lock);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostPathStreams& hs = per_device[dev];
  if (hs.in == nullptr && cudaStreamCreateWithFlags(&hs.in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  if (hs.out == nullptr && cudaStreamCreateWithFlags(&hs.out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
  return &hs;
}
constexpr int kHostPathMaxChunks = 16;   // two status words per chunk fit the arena's 256-byte status region
}  // namespace

// The heads are independent problems, so the host path runs them as a pipeline of head groups:
// group c+1 is copied in (copy stream) while group c is selected and attended (the caller's stream)
// and the output of group c-1 is copied out (second copy stream); host->device and device->host
// copies use different copy engines.  Each group's two status words are kept in the arena.
int sparkattn_attention_host(const sparkattn_shape_t* shape, int32_t dtype, const void* q_host,
                             const void* k_host, const void* v_host, int32_t topk, void* out_host,
                             int32_t* kept_idx_host, void* arena, size_t arena_bytes, void* cuda_stream) {
  int rc = check_shape(shape);
  if (rc != SPARKATTN_OK) return rc;
  if (!q_host || !k_host || !v_host || !out_host || !arena) return SPARKATTN_E_INVALID_ARG;
  if (dtype != SPARKATTN_BF16 && dtype != SPARKATTN_FP8_E4M3) return SPARKATTN_E_INVALID_ARG;
  const int nb = num_blocks(shape);
  if (topk < 1 || topk > nb) return SPARKATTN_E_INVALID_ARG;
  if (!aligned256(arena)) return SPARKATTN_E_MISALIGNED;
  // a head group never spans two batch entries, so the batch count bounds the number of groups from below
  if (shape->B > kHostPathMaxChunks) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  sparkattn_shape_t s = *shape;  // host tensors are contiguous
  s.stride_n = s.d; s.stride_h = (int64_t)s.N * s.d; s.stride_b = (int64_t)s.H * s.N * s.d;
  const Arena a = plan_arena(s, dtype, topk);
  if (arena_bytes < a.total) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  HostPathStreams* hs = host_path_streams();
  if (hs == nullptr) return SPARKATTN_E_CUDA;
  char* base = static_cast<char*>(arena);

  // head groups: about 8 per call, never across a batch boundary
  int heads_per_chunk = (s.H + 7) / 8;
  while (heads_per_chunk < s.H && (int64_t)s.B * ((s.H + heads_per_chunk - 1) / heads_per_chunk) > kHostPathMaxChunks)
    ++heads_per_chunk;
  struct Chunk { int b, h0, hc; };
  Chunk chunks[kHostPathMaxChunks];
  int n_chunks = 0;
  for (int b = 0; b < s.B; ++b)
    for (int h0 = 0; h0 < s.H; h0 += heads_per_chunk) chunks[n_chunks++] = Chunk{b, h0, min(heads_per_chunk, s.H - h0)};

  cudaEvent_t ev_start = nullptr, ev_in[kHostPathMaxChunks] = {}, ev_done[kHostPathMaxChunks] = {}, ev_out = nullptr;
  auto destroy_events = [&]() {
    if (ev_start) cudaEventDestroy(ev_start);
    if (ev_out) cudaEventDestroy(ev_out);
    for (int c = 0; c < n_chunks; ++c) {
      if (ev_in[c]) cudaEventDestroy(ev_in[c]);
      if (ev_done[c]) cudaEventDestroy(ev_done[c]);
    }
  };
  // after an enqueue error: let what is already in flight finish before the events go
  auto fail = [&](int code) {
    cudaStreamSynchronize(hs->in); cudaStreamSynchronize(stream); cudaStreamSynchronize(hs->out);
    destroy_events();
    return code;
  };
  bool ev_ok = cudaEventCreateWithFlags(&ev_start, cudaEventDisableTiming) == cudaSuccess &&
               cudaEventCreateWithFlags(&ev_out, cudaEventDisableTiming) == cudaSuccess;
  for (int c = 0; ev_ok && c < n_chunks; ++c)
    ev_ok = cudaEventCreateWithFlags(&ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ev_done[c], cudaEventDisableTiming) == cudaSuccess;
  if (!ev_ok) { destroy_events(); return SPARKATTN_E_CUDA; }

  // the copy streams start after whatever the caller already queued on its stream
  if (cudaEventRecord(ev_start, stream) != cudaSuccess || cudaStreamWaitEvent(hs->in, ev_start, 0) != cudaSuccess ||
      cudaStreamWaitEvent(hs->out, ev_start, 0) != cudaSuccess)
    return fail(SPARKATTN_E_CUDA);
  if (cudaMemsetAsync(base + a.status, 0, 256, stream) != cudaSuccess) return fail(SPARKATTN_E_CUDA);

  int32_t* idx_all = reinterpret_cast<int32_t*>(base + a.idx);
  int32_t* cnt_all = reinterpret_cast<int32_t*>(base + a.cnt);
  int32_t* status_dev = reinterpret_cast<int32_t*>(base + a.status);
  for (int c = 0; c < n_chunks; ++c) {
    const Chunk& ch = chunks[c];
    const size_t elem_off = ((size_t)ch.b * s.H + ch.h0) * (size_t)s.N * s.d;   // elements before the group
    const size_t bytes = (size_t)ch.hc * s.N * s.d * 2;
    const size_t row_off = ((size_t)ch.b * s.H + ch.h0) * nb;                   // (head, block) rows before it
    if (cudaMemcpyAsync(base + a.q + elem_off * 2, static_cast<const char*>(q_host) + elem_off * 2, bytes,
                        cudaMemcpyHostToDevice, hs->in) != cudaSuccess ||
        cudaMemcpyAsync(base + a.k + elem_off * 2, static_cast<const char*>(k_host) + elem_off * 2, bytes,
                        cudaMemcpyHostToDevice, hs->in) != cudaSuccess ||
        cudaMemcpyAsync(base + a.v + elem_off * 2, static_cast<const char*>(v_host) + elem_off * 2, bytes,
                        cudaMemcpyHostToDevice, hs->in) != cudaSuccess ||
        cudaEventRecord(ev_in[c], hs->in) != cudaSuccess || cudaStreamWaitEvent(stream, ev_in[c], 0) != cudaSuccess)
      return fail(SPARKATTN_E_CUDA);

    sparkattn_shape_t cs = s;      // one batch entry, the group's heads, strides of the full tensors
    cs.B = 1; cs.H = ch.hc;
    int32_t* idx = idx_all + row_off * topk;
    int32_t* cnt = cnt_all + row_off;
    rc = sparkattn_select(&cs, base + a.q + elem_off * 2, base + a.k + elem_off * 2, topk, idx, cnt, base + a.ws_sel,
                          select_workspace_bytes(cs), cuda_stream);
    if (rc != SPARKATTN_OK) return fail(rc);
    const void *fq = base + a.q + elem_off * 2, *fk = base + a.k + elem_off * 2, *fv = base + a.v + elem_off * 2;
    const float *sq = nullptr, *sk = nullptr, *sv = nullptr;
    if (dtype == SPARKATTN_FP8_E4M3) {
      const size_t tensor_off[3] = {a.q, a.k, a.v}, code_off[3] = {a.cq, a.ck, a.cv}, scale_off[3] = {a.sq, a.sk, a.sv};
      for (int i = 0; i < 3; ++i) {
        rc = sparkattn_quant_fp8(&cs, base + tensor_off[i] + elem_off * 2,
                                 reinterpret_cast<uint8_t*>(base + code_off[i] + elem_off),
                                 reinterpret_cast<float*>(base + scale_off[i]) + row_off, 0, cuda_stream);
        if (rc != SPARKATTN_OK) return fail(rc);
      }
      fq = base + a.cq + elem_off; fk = base + a.ck + elem_off; fv = base + a.cv + elem_off;
      sq = reinterpret_cast<const float*>(base + a.sq) + row_off;
      sk = reinterpret_cast<const float*>(base + a.sk) + row_off;
      sv = reinterpret_cast<const float*>(base + a.sv) + row_off;
    }
    rc = sparkattn_fwd(&cs, dtype, fq, fk, fv, sq, sk, sv, idx, cnt, topk, base + a.out + elem_off * 2, nullptr,
                       base + a.ws_fwd, fwd_workspace_bytes(cs, topk), cuda_stream);
    if (rc != SPARKATTN_OK) return fail(rc);
    // the next group reuses both workspaces: keep this group's status words
    if (cudaMemcpyAsync(status_dev + 2 * c, base + a.ws_sel, 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(status_dev + 2 * c + 1, base + a.ws_fwd, 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
        cudaEventRecord(ev_done[c], stream) != cudaSuccess || cudaStreamWaitEvent(hs->out, ev_done[c], 0) != cudaSuccess)
      return fail(SPARKATTN_E_CUDA);
    if (cudaMemcpyAsync(static_cast<char*>(out_host) + elem_off * 2, base + a.out + elem_off * 2, bytes,
                        cudaMemcpyDeviceToHost, hs->out) != cudaSuccess)
      return fail(SPARKATTN_E_CUDA);
    if (kept_idx_host != nullptr &&
        cudaMemcpyAsync(kept_idx_host + row_off * topk, idx, (size_t)ch.hc * nb * topk * 4, cudaMemcpyDeviceToHost,
                        hs->out) != cudaSuccess)
      return fail(SPARKATTN_E_CUDA);
  }
  // the caller's stream ends after the last copy out
  if (cudaEventRecord(ev_out, hs->out) != cudaSuccess || cudaStreamWaitEvent(stream, ev_out, 0) != cudaSuccess)
    return fail(SPARKATTN_E_CUDA);
  int32_t st[2 * kHostPathMaxChunks] = {};
  if (cudaMemcpyAsync(st, status_dev, sizeof(int32_t) * 2 * n_chunks, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return fail(SPARKATTN_E_CUDA);
  if (cudaStreamSynchronize(stream) != cudaSuccess) return fail(SPARKATTN_E_CUDA);
  destroy_events();
  for (int i = 0; i < 2 * n_chunks; ++i)
    if (st[i] != 0) return st[i];
  return SPARKATTN_OK;
}

}  // extern "C"
