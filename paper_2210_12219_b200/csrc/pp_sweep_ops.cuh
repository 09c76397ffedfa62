// Device helpers shared by the register-tiled sweep kernels: packed 16-bit min/max, shuffles that
// shift +inf in, and the slow path of the final-state bookkeeping.
#pragma once
#include "pp_internal.cuh"

namespace pp {

constexpr uint32_t kInf2 = 0xFFFFFFFFu;  // two +inf ranks

__device__ __forceinline__ uint32_t vmin2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("min.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t vmax2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
// three-input packed minimum: one issue slot where two two-input minima would take two
__device__ __forceinline__ uint32_t vmin3(uint32_t a, uint32_t b, uint32_t c) { return __vimin3_u16x2(a, b, c); }
// shuffle up by delta (<= 31) lanes, +inf shifted in from below lane 0
__device__ __forceinline__ uint32_t shfl_up_inf(uint32_t x, int delta)
{
    uint32_t y;
    asm volatile("{ .reg .pred p; shfl.sync.up.b32 %0|p, %1, %2, 0, 0xffffffff; @!p mov.b32 %0, 0xffffffff; }"
                 : "=r"(y) : "r"(x), "r"(delta));
    return y;
}
// acc = min(acc, x shifted up by delta lanes); lanes without a source keep acc
__device__ __forceinline__ void min_shfl_up(uint32_t &acc, uint32_t x, int delta)
{
    asm volatile("{ .reg .pred p; .reg .b32 t; shfl.sync.up.b32 t|p, %1, %2, 0, 0xffffffff; @p min.u16x2 %0, %0, t; }"
                 : "+r"(acc) : "r"(x), "r"(delta));
}

// Slow path of the final-state bookkeeping, kept out of line so that the common case is a
// compare and a branch.
static __device__ __noinline__ unsigned long long offer_final(unsigned long long *best,
                                                              unsigned long long best_seen, uint32_t val,
                                                              int level, uint32_t S2, int w)
{
    const unsigned long long key = pack_best(val, level, S2, w);
    if (key < best_seen) {
        atomicMin(best, key);
        return key;
    }
    return best_seen;
}

}  // namespace pp
