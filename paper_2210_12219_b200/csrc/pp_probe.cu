// Issue-rate probe for the instructions the (min,max) sweep is made of (see pp_debug_minmax_rate in
// pp.h).  One block of 1024 threads per SM runs unrolled chains of one packed 16-bit min/max form
// on registers only and reads the SM's clock before and after; the result is warp instructions
// per clock per SM, the figure the ALU bound of the roofline is derived from.
#include "pp_internal.cuh"

namespace pp {

namespace {

constexpr int kProbeThreads = 1024;
constexpr int kProbeChains = 8;    // independent accumulators per thread
constexpr int kProbeUnroll = 8;    // instructions per accumulator per loop trip

// OP 0: two-input forms, minimum and maximum in turn (a chain of minima alone could be merged into
// three-input instructions by the assembler and would then count double); OP 1 / OP 2: the
// three-input minimum / maximum, one instruction each on this architecture.
template <int OP>
__device__ __forceinline__ uint32_t probe_op(uint32_t a, uint32_t b, uint32_t c, int u)
{
    uint32_t r;
    if (OP == 0) {
        if (u & 1) asm volatile("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        else asm volatile("min.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(c));
    } else if (OP == 1) {
        r = __vimin3_u16x2(a, b, c);
    } else {
        r = __vimax3_u16x2(a, b, c);
    }
    return r;
}

template <int OP>
__global__ void __launch_bounds__(kProbeThreads, 1)
k_probe(int iters, uint32_t seed, long long *cycles, uint32_t *sink)
{
    uint32_t acc[kProbeChains];
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) acc[i] = seed * (threadIdx.x + 1) + i * 0x10003u;
    const uint32_t b = seed ^ 0x5a5a1234u, c = seed + 0x00070009u;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        const uint32_t bi = b + (uint32_t)it * 0x00010001u;  // operands change from trip to trip
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u)
#pragma unroll
            for (int i = 0; i < kProbeChains; ++i) acc[i] = probe_op<OP>(acc[i], bi + u, c + i, u);
    }
    __syncthreads();
    const long long t1 = clock64();
    uint32_t x = 0;
#pragma unroll
    for (int i = 0; i < kProbeChains; ++i) x ^= acc[i];
    if (x == 0x12345u) sink[0] = x;  // keeps the chains alive
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

}  // namespace

cudaError_t launch_probe(int op, int iters, int blocks, long long *cycles, uint32_t *sink, cudaStream_t s)
{
    switch (op) {
        case 0: k_probe<0><<<blocks, kProbeThreads, 0, s>>>(iters, 0x01020304u, cycles, sink); break;
        case 1: k_probe<1><<<blocks, kProbeThreads, 0, s>>>(iters, 0x01020304u, cycles, sink); break;
        case 2: k_probe<2><<<blocks, kProbeThreads, 0, s>>>(iters, 0x01020304u, cycles, sink); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

double probe_instr_per_block(int iters)
{
    return (double)iters * kProbeUnroll * kProbeChains * (kProbeThreads / 32);
}

}  // namespace pp
