// The generic popcount-level sweep, and the final choice + backtrack.
//
// State (S, v, c): layers 0..c are placed on exactly the nodes of S, one segment each, the
// last segment on v ending at layer c.  Its value is the smallest bottleneck (Eq. 2) any such
// partial plan can have, held as a rank (see pp_internal.cuh).
//   |S| = 1 :  value 0 if layers 0..c fit on v, else +inf
//   else    :  dp[S'][w][c'] = min over c in [lo_w(c'), c'-1] of g[c],
//              g[c] = min over v in S = S'\{w} of max(dp[S][v][c], gamma[c][v][w])
// Every target row (S', w) has exactly one source mask S'\{w}, so a block that owns a source
// mask writes rows nobody else writes: no atomics on the table, no write races.
#include "pp_internal.cuh"

namespace pp {

template <typename T>
__device__ __forceinline__ void offer_best(const Dev &d, T val, uint32_t mask, int v)
{
    const T kInf = (T)~(T)0;
    if (val == kInf) return;
    unsigned long long key = pack_best((uint32_t)val, __popc(mask), mask, v);
    // read first: almost every offer loses, and a plain load is far cheaper than an atomic
    if (key < *reinterpret_cast<volatile unsigned long long *>(d.best)) atomicMin(d.best, key);
}

// Generic sweep of one level: one block per source mask S of popcount level-1.  Works for any
// L, k within the limits and both element types; values and ranks are read from global memory
// (they stay in L1/L2), g rows live in shared memory, each output scans its window directly.
template <typename T>
__global__ void k_sweep_generic(Dev d, int level)
{
    extern __shared__ unsigned char smem_raw[];
    const T kInf = (T)~(T)0;
    T *sg = reinterpret_cast<T *>(smem_raw);  // [nw][Lpad]
    const T *table = reinterpret_cast<const T *>(d.table);
    T *table_w = reinterpret_cast<T *>(d.table);
    const T *rank = reinterpret_cast<const T *>(d.rank);
    const int k = d.k, L = d.L, Lpad = d.Lpad;
    const uint32_t S = d.masks[d.level_off[level - 1] + blockIdx.x];
    const uint32_t full = (k == 32) ? 0xFFFFFFFFu : ((1u << k) - 1u);
    const uint32_t comp = full & ~S;
    const int nw = __popc(comp);

    // g[c] for every target node w not in S
    for (int item = threadIdx.x; item < nw * L; item += blockDim.x) {
        int wi = item / L, c = item - wi * L;
        int w = __fns(comp, 0, wi + 1);
        T g = kInf;
        for (uint32_t rem = S; rem; rem &= rem - 1) {
            int v = __ffs(rem) - 1;
            const size_t ia = ((size_t)S * k + v) * Lpad + c, ib = ((size_t)w * k + v) * Lpad + c;
            if (!PP_IN_BOUNDS(d, ia, d.table_elems) || !PP_IN_BOUNDS(d, ib, d.rank_elems)) continue;
            T a = table[ia];
            T b = rank[ib];
            T m = a > b ? a : b;
            g = m < g ? m : g;
        }
        sg[wi * Lpad + c] = g;
    }
    __syncthreads();
    // window minimum and write-out; pads of each row are set to +inf
    for (int item = threadIdx.x; item < nw * Lpad; item += blockDim.x) {
        int wi = item / Lpad, c2 = item - wi * Lpad;
        int w = __fns(comp, 0, wi + 1);
        T best = kInf;
        if (c2 < L) {
            int lo = d.lo[w * L + c2];
            for (int c = lo; c < c2; ++c) {
                T x = sg[wi * Lpad + c];
                best = x < best ? x : best;
            }
        }
        uint32_t S2 = S | (1u << w);
        const size_t io = ((size_t)S2 * k + w) * Lpad + c2;
        if (PP_IN_BOUNDS(d, io, d.table_elems)) table_w[io] = best;
        if (c2 == L - 1) offer_best<T>(d, best, S2, w);
    }
}

cudaError_t launch_sweep_generic(const Dev &d, int level, cudaStream_t s)
{
    // host mirrors level_off: masks of popcount j number C(k, j)
    unsigned long long n = 1;
    for (int i = 0; i < level - 1; ++i) n = n * (unsigned)(d.k - i) / (unsigned)(i + 1);
    int nw = d.k - (level - 1);
    size_t sm = (size_t)nw * d.Lpad * d.elem;
    cudaError_t e;
    if (d.elem == 2) {
        e = cudaFuncSetAttribute(k_sweep_generic<uint16_t>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        if (e != cudaSuccess) return e;
        k_sweep_generic<uint16_t><<<(unsigned)n, 128, sm, s>>>(d, level);
    } else {
        e = cudaFuncSetAttribute(k_sweep_generic<uint32_t>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        if (e != cudaSuccess) return e;
        k_sweep_generic<uint32_t><<<(unsigned)n, 128, sm, s>>>(d, level);
    }
    return cudaGetLastError();
}

// ---- final choice and backtrack ---------------------------------------------------------
// One block.  The best final state was collected by offer_best during the sweep.  Walking
// back from (S', w, c'), the predecessor is the lowest c, then the lowest v, among
// v in S'\{w}, c in [lo_w(c'), c'-1] with max(dp[S'\{w}][v][c], gamma[c][v][w]) <= beta*.
// Warp i scans the candidates of the i-th node of S'\{w} in ascending c and stops at its first hit.
template <typename T>
__global__ void __launch_bounds__(1024) k_finalize(Dev d, pp_solution *out)
{
    __shared__ unsigned int s_key[32];
    __shared__ unsigned int s_pick;
    asm volatile("griddepcontrol.wait;" ::: "memory");  // a no-op unless launched as a dependent
    const T *table = reinterpret_cast<const T *>(d.table);
    const T *rank = reinterpret_cast<const T *>(d.rank);
    const int k = d.k, L = d.L, Lpad = d.Lpad;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const unsigned long long key = *reinterpret_cast<volatile unsigned long long *>(d.best);

    if (tid < PP_MAX_K) {
        out->cuts[tid] = -1;
        out->placement[tid] = -1;
    }
    if (key == kNoBest) {
        if (tid == 0) {
            out->beta_ms = __longlong_as_double(0x7FF0000000000000ll);
            out->status = PP_INFEASIBLE;
            out->m = 0;
        }
        return;
    }
    const uint32_t rstar = (uint32_t)(key >> 30);
    const int m = (int)((key >> 25) & 31);
    uint32_t S = (uint32_t)((key >> 5) & 0xFFFFF);
    int w = (int)(key & 31);

    // beta* as a double: an entry that carries the winning rank (equal ranks hold equal doubles)
    if (tid == 0) {
        out->beta_ms = rstar != 0 ? d.gu[d.inv[rstar]] : 0.0;
        out->status = PP_OK;
        out->m = m;
    }

    __syncthreads();  // the -1 fill above is complete before plan entries are written
    int c2 = L - 1;
    for (int j = m - 1; j >= 0; --j) {
        if (tid == 0) {
            out->placement[j] = w;
            if (j < m - 1) out->cuts[j] = c2;
        }
        if (j == 0) break;
        const uint32_t P = S & ~(1u << w);
        const int lo = d.lo[w * L + c2];
        const int np = __popc(P);
        unsigned int bestk = 0xFFFFFFFFu;
        for (int vi = wid; vi < np; vi += (int)(blockDim.x >> 5)) {
            const int v = __fns(P, 0, vi + 1);
            const T *trow = table + ((size_t)P * k + v) * Lpad;
            const T *rrow = rank + ((size_t)w * k + v) * Lpad;
            for (int c0 = lo; c0 < c2; c0 += 32) {
                const int c = c0 + lane;
                bool hit = false;
                if (c < c2 && PP_IN_BOUNDS(d, ((size_t)P * k + v) * Lpad + c, d.table_elems) &&
                    PP_IN_BOUNDS(d, ((size_t)w * k + v) * Lpad + c, d.rank_elems)) {
                    const T a = trow[c];
                    const T b = rrow[c];
                    const T mx = a > b ? a : b;
                    hit = (uint32_t)mx <= rstar && mx != (T)~(T)0;
                }
                const unsigned int hits = __ballot_sync(0xFFFFFFFFu, hit);
                if (hits) {
                    const unsigned int kk = ((unsigned)(c0 + __ffs(hits) - 1) << 5) | (unsigned)v;
                    bestk = kk < bestk ? kk : bestk;
                    break;
                }
            }
        }
        if (lane == 0) s_key[wid] = bestk;
        __syncthreads();
        if (wid == 0) {
            unsigned int x = (lane < (int)(blockDim.x >> 5)) ? s_key[lane] : 0xFFFFFFFFu;
            for (int o = 16; o; o >>= 1) {
                unsigned int other = __shfl_xor_sync(0xFFFFFFFFu, x, o);
                x = other < x ? other : x;
            }
            if (lane == 0) s_pick = x;
        }
        __syncthreads();
        const unsigned int pick = s_pick;
        if (pick == 0xFFFFFFFFu) {  // cannot happen on a consistent table; report, do not trap
            if (tid == 0) {
                atomicExch(d.err, kErrBacktrack);
                out->status = PP_ERR_CUDA;  // readers of the record must not take a half-written plan for a result
            }
            return;
        }
        S = P;
        w = (int)(pick & 31u);
        c2 = (int)(pick >> 5);
        __syncthreads();
    }
}

cudaError_t launch_finalize(const Dev &d, pp_solution *out, cudaStream_t s, bool dependent)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(1024);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return d.elem == 2 ? cudaLaunchKernelEx(&cfg, k_finalize<uint16_t>, d, out)
                       : cudaLaunchKernelEx(&cfg, k_finalize<uint32_t>, d, out);
}

}  // namespace pp
