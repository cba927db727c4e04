// sparkattn_select_noalloc: block selection for callers that cannot allocate.
//
// Some hosts of this library run where device allocation is off limits at call
// time: inside a latency-critical serving loop whose memory was carved up at
// start-up, under an allocator that forbids growth after initialisation, or in
// a plugin that is handed input and output buffers and nothing else.  The
// regular sparkattn_select needs a caller-provided workspace for its pooled
// block means; this variant keeps that scratch in a fixed array that is part
// of the library image instead, so the caller passes inputs and outputs only.
//
// The array costs kNoAllocScratchBytes of device memory on every GPU that
// loads the library, for the life of the process.  All calls share it: it
// still holds the previous call's pooled means when a call starts (the status
// header is cleared per call; the pooled means are fully overwritten before
// they are read), and two calls whose kernels overlap on the GPU (different
// streams, or different host threads) would race on it.
#include <mutex>

#include "common.cuh"
#include "launch.h"

namespace sparkattn {

constexpr size_t kNoAllocScratchBytes = 32u << 20;  // 32 MiB: holds the 40-head, 75,600-token, d=128 case (24.6 MB)

// File-scope device array.  In host code this name is only a handle for the
// runtime's symbol table, never a device address: the address each device
// gave it is fetched once with cudaGetSymbolAddress and cached below.
static __device__ __align__(256) unsigned char g_select_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_mu;
static void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device (set-up on first use per device).
static int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return SPARKATTN_E_NO_DEVICE;
  if (dev < 0 || dev >= kMaxDevices) return SPARKATTN_E_UNSUPPORTED_SHAPE;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_select_scratch) != cudaSuccess || ptr == nullptr) return SPARKATTN_E_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return SPARKATTN_OK;
}

}  // namespace sparkattn

using namespace sparkattn;

extern "C" {

size_t sparkattn_select_noalloc_max_bytes(void) { return kNoAllocScratchBytes; }

int sparkattn_select_noalloc(const sparkattn_shape_t* shape, const void* q_bf16, const void* k_bf16, int32_t topk,
                             int32_t* kept_idx, int32_t* kept_cnt, void* cuda_stream) {
  // Scratch this shape needs (0 if the shape itself is invalid: sparkattn_select below names that error).
  const size_t need = sparkattn_workspace_bytes(shape, 0, topk);
  if (need > kNoAllocScratchBytes) return SPARKATTN_E_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != SPARKATTN_OK) return rc;
  return sparkattn_select(shape, q_bf16, k_bf16, topk, kept_idx, kept_cnt, scratch, kNoAllocScratchBytes,
                          cuda_stream);
}

int sparkattn_select_noalloc_status(void* cuda_stream) {
  void* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != SPARKATTN_OK) return rc;
  return sparkattn_read_status(scratch, cuda_stream);
}

}  // extern "C"
