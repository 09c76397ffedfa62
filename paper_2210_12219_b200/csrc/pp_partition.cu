// Partition stage of the paper's heuristic (Section 3.2.1, Eq. 6-7, Algorithm 1), many chains per
// launch: split a chain of L cut points into contiguous partitions that each fit the capacity
// kappa of a node, minimising the sum of the weights of the points a partition ends with (the
// tensor that crosses the cut; the last partition sends nothing).
//
// The paper walks an explicit graph of all feasible partitions with a memo per last point.  Here
// the same optimum is a chain recurrence over suffixes with the sliding memory window of the
// exact search:   F[i] = min over e in [i, hi(i)] of G[e],   G[e] = weight[e] + F[e + 1],  G[L-1] = 0,
// where hi(i) is the last point such that points i..hi(i) fit.  Values carry the number of
// partitions in their low bits, (cost << 11 | partitions), so that one unsigned minimum applies the
// tie rule "smaller cost, then fewer partitions"; walking forward from point 0 and always taking
// the earliest e that attains F[i] gives the lexicographically smallest cut list among those.
//
// Two kernels.  One warp per chain (any length, small batches): the recurrence is L dependent steps,
// each a minimum over a window that the lanes scan together; prefix sums of the memory and the G
// values live in the warp's slice of shared memory, the weights pass through registers 32 at a time.
// One lane per chain (chains of up to 64 points, 8192 chains or more): see k_partition_lanes.
#include "pp_internal.cuh"

namespace pp {

namespace {

constexpr int kPartWarps = 4;
constexpr unsigned long long kInfCost = ~0ull;
constexpr int kPartsBits = 11;  // partitions <= PP_MAX_L = 1024 < 2^11

__device__ __forceinline__ unsigned long long warp_min_u64(unsigned long long x)
{
    for (int o = 16; o; o >>= 1) {
        const unsigned long long y = __shfl_xor_sync(0xFFFFFFFFu, x, o);
        x = y < x ? y : x;
    }
    return x;
}

__global__ void __launch_bounds__(kPartWarps * 32)
k_partition_minsum(int64_t B, int L, int cap_seg, const uint64_t *__restrict__ weight,
                   const uint64_t *__restrict__ mem, const uint64_t *__restrict__ kappa,
                   uint64_t *__restrict__ o_cost, int32_t *__restrict__ o_m, int32_t *__restrict__ o_cuts,
                   uint64_t *__restrict__ o_sizes, int8_t *__restrict__ o_status)
{
    extern __shared__ unsigned long long smem_u64[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long *M = smem_u64 + (size_t)wid * (2 * L + 1);  // [L + 1] prefix sums of the memory
    unsigned long long *G = M + (L + 1);                           // [L]
    for (int64_t b = (int64_t)blockIdx.x * kPartWarps + wid; b < B; b += (int64_t)gridDim.x * kPartWarps) {
        const uint64_t *w = weight + b * L, *mm = mem + b * L;
        const unsigned long long cap = kappa[b];
        __syncwarp();
        // prefix sums, 32 points at a time; a wrapping sum or a weight beyond the limit voids the chain
        bool bad = false;
        unsigned long long carry = 0;
        if (lane == 0) M[0] = 0;
        for (int base = 0; base < L; base += 32) {
            const int i = base + lane;
            unsigned long long x = i < L ? mm[i] : 0ull;
            if (i < L && w[i] >= PP_MAX_BITS) bad = true;
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
                if (lane >= o) {
                    if (y > ~0ull - x) bad = true;
                    x += y;
                }
            }
            if (x > ~0ull - carry) bad = true;
            x += carry;
            if (i < L) M[i + 1] = x;
            carry = __shfl_sync(0xFFFFFFFFu, x, 31);
        }
        bad = __any_sync(0xFFFFFFFFu, bad);
        int32_t *cuts = o_cuts ? o_cuts + b * cap_seg : nullptr;
        uint64_t *sizes = o_sizes ? o_sizes + b * cap_seg : nullptr;
        for (int j = lane; j < cap_seg; j += 32) {
            if (cuts) cuts[j] = -1;
            if (sizes) sizes[j] = 0;
        }
        if (bad) {
            if (lane == 0) {
                o_cost[b] = 0;
                o_m[b] = 0;
                o_status[b] = (int8_t)PP_ERR_LIMIT;
            }
            continue;
        }
        __syncwarp();
        // backward recurrence
        unsigned long long F = kInfCost, wchunk = 0;
        int hi = L - 1;
        for (int i = L - 1; i >= 0; --i) {
            if (i == L - 1 || (i & 31) == 31) {  // weights of points i-31 .. i (i - 1 is the one needed next)
                const int e = (i & ~31) + lane;
                wchunk = e < L ? w[e] : 0ull;
            }
            if (i == L - 1) {
                if (lane == 0) G[L - 1] = 1ull;  // cost 0, one partition
                __syncwarp();
            }
            while (hi >= i && M[hi + 1] - M[i] > cap) --hi;
            unsigned long long best = kInfCost;
            for (int e = i + lane; e <= hi; e += 32) {
                const unsigned long long g = G[e];
                best = g < best ? g : best;
            }
            F = warp_min_u64(best);
            if (i > 0) {
                const unsigned long long wi = __shfl_sync(0xFFFFFFFFu, wchunk, (i - 1) & 31);
                // the chunk that holds point i - 1 is the current one unless i is a multiple of 32
                unsigned long long wprev = wi;
                if ((i & 31) == 0) wprev = w[i - 1];
                if (lane == 0) G[i - 1] = F == kInfCost ? kInfCost : F + (wprev << kPartsBits) + 1ull;
                __syncwarp();
            }
        }
        if (F == kInfCost) {
            if (lane == 0) {
                o_cost[b] = 0;
                o_m[b] = 0;
                o_status[b] = (int8_t)PP_INFEASIBLE;
            }
            continue;
        }
        const int parts = (int)(F & ((1ull << kPartsBits) - 1ull));
        if (lane == 0) {
            o_cost[b] = F >> kPartsBits;
            o_m[b] = parts;
            o_status[b] = parts > cap_seg + 1 ? (int8_t)PP_ERR_LIMIT : (int8_t)PP_OK;  // cuts do not fit the caller's rows
        }
        if (parts > cap_seg + 1) continue;
        // forward walk: the earliest point that attains the optimum of the suffix
        unsigned long long target = F;
        int i = 0, nc = 0;
        hi = -1;
        for (;;) {
            if (hi < i) hi = i;
            while (hi + 1 < L && M[hi + 2] - M[i] <= cap) ++hi;
            int found = -1;
            for (int base = i; base <= hi && found < 0; base += 32) {
                const int e = base + lane;
                const unsigned int hits = __ballot_sync(0xFFFFFFFFu, e <= hi && G[e] == target);
                if (hits) found = base + __ffs(hits) - 1;
            }
            if (found < 0 || found == L - 1) break;  // found < 0 cannot happen on a consistent table
            const unsigned long long wf = w[found];
            if (lane == 0) {
                if (cuts) cuts[nc] = found;
                if (sizes) sizes[nc] = wf;
            }
            ++nc;
            target = target - (wf << kPartsBits) - 1ull;
            i = found + 1;
        }
    }
}

// The same recurrence with one chain per lane, for short chains in bulk: every lane of a warp walks
// its own chain through the same loop, so the control of a step is paid once per 32 chains, and the
// window minimum needs no reduction across lanes.  A lane's prefix sums and G values sit in its own
// column of shared memory, element (i, lane) at word pair (i * 32 + lane): whatever index a lane
// uses, it stays in its own banks.  Same tie rules, same outputs.
constexpr int kLaneWarps = 2;
constexpr int kLaneMaxL = 64;   // (2 L + 1) * 256 bytes of shared memory per warp
constexpr int kLaneMinB = 8192;  // below this the warp-per-chain kernel has more warps to hide the steps' latency behind

__global__ void __launch_bounds__(kLaneWarps * 32)
k_partition_lanes(int64_t B, int L, int cap_seg, const uint64_t *__restrict__ weight,
                  const uint64_t *__restrict__ mem, const uint64_t *__restrict__ kappa,
                  uint64_t *__restrict__ o_cost, int32_t *__restrict__ o_m, int32_t *__restrict__ o_cuts,
                  uint64_t *__restrict__ o_sizes, int8_t *__restrict__ o_status)
{
    extern __shared__ unsigned long long smem_u64[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long *M = smem_u64 + (size_t)wid * (2 * L + 1) * 32 + lane;  // M[i * 32]: memory of points 0..i-1
    unsigned long long *G = M + (size_t)(L + 1) * 32;                          // G[e * 32]
    const int64_t groups = (B + 31) >> 5;
    for (int64_t g = (int64_t)blockIdx.x * kLaneWarps + wid; g < groups; g += (int64_t)gridDim.x * kLaneWarps) {
        const int64_t b0 = g * 32, b = b0 + lane;
        const bool act = b < B;
        const int64_t rows = (B - b0 < 32 ? B - b0 : 32) * (int64_t)cap_seg;
        // the 32 chains' output rows are one contiguous stretch: cleared by the warp together
        for (int64_t j = lane; j < rows; j += 32) {
            if (o_cuts) o_cuts[b0 * cap_seg + j] = -1;
            if (o_sizes) o_sizes[b0 * cap_seg + j] = 0;
        }
        __syncwarp();
        const uint64_t *w = weight + (act ? b : b0) * L, *mm = mem + (act ? b : b0) * L;
        const unsigned long long cap = kappa[act ? b : b0];
        bool bad = false;
        unsigned long long acc = 0;
        M[0] = 0;
        for (int i = 0; i < L; ++i) {
            const unsigned long long x = mm[i];
            if (w[i] >= PP_MAX_BITS) bad = true;
            if (x > ~0ull - acc) bad = true;  // the 64-bit sum would wrap
            acc += x;
            M[(size_t)(i + 1) * 32] = acc;
        }
        // backward recurrence
        unsigned long long F = kInfCost;
        int hi = L - 1;
        G[(size_t)(L - 1) * 32] = 1ull;  // cost 0, one partition
        unsigned long long wprev = L > 1 ? w[L - 2] : 0ull;
        for (int i = L - 1; i >= 0; --i) {
            const unsigned long long wcur = wprev;          // weight of point i - 1
            if (i >= 2) wprev = w[i - 2];                   // asked for one step ahead
            const unsigned long long Mi = M[(size_t)i * 32];
            while (hi >= i && M[(size_t)(hi + 1) * 32] - Mi > cap) --hi;
            unsigned long long best = kInfCost;
            for (int e = i; e <= hi; ++e) {
                const unsigned long long x = G[(size_t)e * 32];
                best = x < best ? x : best;
            }
            F = best;
            if (i > 0) G[(size_t)(i - 1) * 32] = F == kInfCost ? kInfCost : F + (wcur << kPartsBits) + 1ull;
        }
        if (!act) continue;
        if (bad || F == kInfCost) {
            o_cost[b] = 0;
            o_m[b] = 0;
            o_status[b] = bad ? (int8_t)PP_ERR_LIMIT : (int8_t)PP_INFEASIBLE;
            continue;
        }
        const int parts = (int)(F & ((1ull << kPartsBits) - 1ull));
        o_cost[b] = F >> kPartsBits;
        o_m[b] = parts;
        o_status[b] = parts > cap_seg + 1 ? (int8_t)PP_ERR_LIMIT : (int8_t)PP_OK;  // cuts do not fit the caller's rows
        if (parts > cap_seg + 1) continue;
        // forward walk: the earliest point that attains the optimum of the suffix
        unsigned long long target = F;
        int i = 0, nc = 0;
        for (;;) {
            int found = -1;
            const unsigned long long Mi = M[(size_t)i * 32];
            for (int e = i; e < L && M[(size_t)(e + 1) * 32] - Mi <= cap; ++e)
                if (G[(size_t)e * 32] == target) {
                    found = e;
                    break;
                }
            if (found < 0 || found == L - 1) break;  // found < 0 cannot happen on a consistent table
            const unsigned long long wf = w[found];
            if (o_cuts) o_cuts[b * cap_seg + nc] = found;
            if (o_sizes) o_sizes[b * cap_seg + nc] = wf;
            ++nc;
            target = target - (wf << kPartsBits) - 1ull;
            i = found + 1;
        }
    }
}

}  // namespace

size_t partition_smem_bytes(int L) { return (size_t)kPartWarps * (2 * (size_t)L + 1) * sizeof(unsigned long long); }

cudaError_t launch_partition_minsum(int64_t B, int L, int cap_seg, const uint64_t *weight, const uint64_t *mem,
                                    const uint64_t *kappa, uint64_t *cost, int32_t *m, int32_t *cuts,
                                    uint64_t *sizes, int8_t *status, cudaStream_t s)
{
    if (B <= 0) return cudaSuccess;
    if (B >= kLaneMinB && L <= kLaneMaxL) {
        const size_t lsm = (size_t)kLaneWarps * (2 * (size_t)L + 1) * 32 * sizeof(unsigned long long);
        cudaError_t el = cudaFuncSetAttribute(k_partition_lanes, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lsm);
        if (el != cudaSuccess) return el;
        const int64_t groups = (B + 31) / 32;
        int64_t lblocks = (groups + kLaneWarps - 1) / kLaneWarps;
        if (lblocks > 148 * 32) lblocks = 148 * 32;
        k_partition_lanes<<<(unsigned)lblocks, kLaneWarps * 32, lsm, s>>>(B, L, cap_seg, weight, mem, kappa, cost, m, cuts,
                                                                           sizes, status);
        return cudaGetLastError();
    }
    const size_t sm = partition_smem_bytes(L);
    cudaError_t e = cudaFuncSetAttribute(k_partition_minsum, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    int64_t blocks = (B + kPartWarps - 1) / kPartWarps;
    const int64_t cap = 148 * 32;
    if (blocks > cap) blocks = cap;
    k_partition_minsum<<<(unsigned)blocks, kPartWarps * 32, sm, s>>>(B, L, cap_seg, weight, mem, kappa, cost, m, cuts,
                                                                     sizes, status);
    return cudaGetLastError();
}

}  // namespace pp
