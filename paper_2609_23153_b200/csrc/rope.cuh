// Rank-truncated rotary rotation of the compensation branch (Sec. 4.1): what the branch's own kernels (comp.cu)
// and the forward kernel's fused gate epilogue (fwd_pipe.cu) share.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "launch.h"

namespace sparkattn {

struct RopeTable {
  int32_t axis[kCompRank / 2];        // 0 = t, 1 = y, 2 = x
  float freq[kCompRank / 2];
  int32_t T, Hg, Wg;
};

// Bytes of the position-major cos / sin table of a (T, Hg, Wg) grid, and the launch that fills it:
// table[(base(axis) + e) * rank/2 + m] = (cos, sin)(e * freq[m]), base(t) = 0, base(y) = T, base(x) = T + Hg.
size_t rope_table_bytes(const int32_t* grid);
void launch_rope_table(const RopeTable& rope, float2* table, cudaStream_t stream);

__device__ __forceinline__ float fast_rcp(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace sparkattn
