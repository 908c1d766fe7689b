// Device-side helpers shared by the copy kernels.
#pragma once

#include <cstdint>

namespace pdkv {

// n / d through one multiply: m = floor(2^32 / d) + 1 (0 stands for d == 1; for a
// power of two the expression below gives 2^32 / d, also exact).  Exact while
// n * d < 2^32, which the planner guarantees for every tile.
__device__ __forceinline__ uint32_t fast_div(uint32_t n, uint32_t m) { return m ? __umulhi(n, m) : n; }
__device__ __forceinline__ uint32_t div_magic(uint32_t d) { return d == 1u ? 0u : 0xFFFFFFFFu / d + 1u; }

}  // namespace pdkv
