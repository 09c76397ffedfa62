// Exact search under the paper's full objective, Eq. 1: the bottleneck of a plan is the largest of
// the compute times of its partitions and the transfer latencies of its cuts (Eq. 2 drops the
// compute times).  Same state space as the main search, dp over (used-node set S, last node v, last
// layer c), with the compute time of the last partition inside the minimum:
//   |S| = 1 :  dp[{v}][v][c] = comp_v(0..c) if layers 0..c fit on v, else +inf
//   else    :  dp[S'][w][c'] = min over c in [lo_w(c'), c'-1] of max(g[c], comp_w(c+1..c')),
//              g[c] = min over v in S'\{w} of max(dp[S'\{w}][v][c], gamma[c][v][w])
// comp_w(first..last) = (sum of the layers' work) / speed[w]: one correctly rounded fp64 division of
// exact integers, like gamma (Eq. 3).  The compute term depends on both ends of the partition, so the
// window minimum does not factor as in the main search: every output scans its window.  Values are
// kept as doubles (there are L*L*k/2 distinct compute times, too many for 16-bit ranks); the table
// of every comp_w(c+1..c') is built once.  One block per source mask, the g rows in shared memory.
// This is the plain kernel family of the build (no register tiling): the objective is an extension,
// not the benchmarked path.
#include "pp_internal.cuh"

namespace pp {

namespace {

__device__ __forceinline__ double dinf() { return __longlong_as_double(0x7FF0000000000000ll); }

// gam[(w*k+v)*L + c], seg[(w*L+c2)*L + c] for c < c2 inside the window, base frontier rows
__global__ void k_ct_tables(CtDev d)
{
    const int k = d.k, L = d.L;
    const int b = blockIdx.x;
    if (b < k * k) {
        const int w = b / k, v = b - w * k;
        const uint32_t link = d.bw[v * k + w];
        for (int c = threadIdx.x; c < L; c += blockDim.x)
            d.gam[(size_t)b * L + c] = (v == w || link == 0) ? dinf() : __ddiv_rn((double)d.bits[c], (double)link);
    } else if (b < k * k + k * L) {
        const int r = b - k * k, w = r / L, c2 = r - w * L;
        const uint32_t sp = d.speed[w];
        for (int c = threadIdx.x; c < L; c += blockDim.x) {
            double x = dinf();
            if (c < c2 && sp != 0 && d.M[c2 + 1] - d.M[c + 1] <= d.cap[w])
                x = __ddiv_rn((double)(d.Wp[c2 + 1] - d.Wp[c + 1]), (double)sp);
            d.seg[(size_t)r * L + c] = x;
        }
    } else {
        const int v = b - k * k - k * L;
        const uint32_t sp = d.speed[v];
        double *row = d.table + ((size_t)(1u << v) * k + v) * L;
        for (int c = threadIdx.x; c < L; c += blockDim.x)
            row[c] = (sp != 0 && d.M[c + 1] <= d.cap[v]) ? __ddiv_rn((double)d.Wp[c + 1], (double)sp) : dinf();
    }
}

__global__ void __launch_bounds__(128) k_ct_level(CtDev d, int level)
{
    extern __shared__ double sg[];  // [nw][L]
    const int k = d.k, L = d.L;
    const uint32_t S = d.masks[d.level_off[level - 1] + blockIdx.x];
    const uint32_t comp = ((1u << k) - 1u) & ~S;
    const int nw = __popc(comp);
    for (int item = threadIdx.x; item < nw * L; item += blockDim.x) {
        const int wi = item / L, c = item - wi * L;
        const int w = __fns(comp, 0, wi + 1);
        double g = dinf();
        for (uint32_t rem = S; rem; rem &= rem - 1) {
            const int v = __ffs(rem) - 1;
            const double a = d.table[((size_t)S * k + v) * L + c];
            const double b = d.gam[((size_t)w * k + v) * L + c];
            const double mx = a > b ? a : b;
            g = mx < g ? mx : g;
        }
        sg[wi * L + c] = g;
    }
    __syncthreads();
    for (int item = threadIdx.x; item < nw * L; item += blockDim.x) {
        const int wi = item / L, c2 = item - wi * L;
        const int w = __fns(comp, 0, wi + 1);
        const double *sw = d.seg + ((size_t)w * L + c2) * L;
        double best = dinf();
        for (int c = c2 - 1; c >= 0; --c) {  // the memory window is a run that ends at c2 - 1: seg is +inf below it
            const double a = sg[wi * L + c], b = sw[c];
            if (b == dinf()) break;
            const double mx = a > b ? a : b;
            best = mx < best ? mx : best;
        }
        d.table[((size_t)(S | (1u << w)) * k + w) * L + c2] = best;
    }
}

// smallest final value (bit pattern of a non-negative double orders like the value), then the
// smallest (popcount, mask, node) among the states that attain it
__global__ void k_ct_best(CtDev d, int pass)
{
    const int k = d.k, L = d.L;
    const uint32_t nm = 1u << k;
    for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r < nm * (uint32_t)k; r += gridDim.x * blockDim.x) {
        const uint32_t S = r / k;
        const int v = r - S * k;
        if (!((S >> v) & 1u) || __popc(S) > L) continue;
        const double x = d.table[(size_t)r * L + (L - 1)];
        if (x == dinf()) continue;
        const unsigned long long bits = (unsigned long long)__double_as_longlong(x);
        if (pass == 0) atomicMin(d.best_val, bits);
        else if (bits == *d.best_val)
            atomicMin(d.best_key, ((unsigned long long)__popc(S) << 25) | ((unsigned long long)S << 5) | (unsigned long long)v);
    }
}

__global__ void __launch_bounds__(256) k_ct_backtrack(CtDev d, pp_solution *out)
{
    __shared__ unsigned int s_key[8];
    __shared__ unsigned int s_pick;
    const int k = d.k, L = d.L, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid < PP_MAX_K) {
        out->cuts[tid] = -1;
        out->placement[tid] = -1;
    }
    const unsigned long long key = *d.best_key;
    if (key == ~0ull) {
        if (tid == 0) {
            out->beta_ms = dinf();
            out->status = PP_INFEASIBLE;
            out->m = 0;
        }
        return;
    }
    const double beta = __longlong_as_double((long long)*d.best_val);
    const int m = (int)((key >> 25) & 31);
    uint32_t S = (uint32_t)((key >> 5) & 0xFFFFF);
    int w = (int)(key & 31), c2 = L - 1;
    if (tid == 0) {
        out->beta_ms = beta;
        out->status = PP_OK;
        out->m = m;
    }
    __syncthreads();
    for (int j = m - 1; j >= 0; --j) {
        if (tid == 0) {
            out->placement[j] = w;
            if (j < m - 1) out->cuts[j] = c2;
        }
        if (j == 0) break;
        const uint32_t P = S & ~(1u << w);
        const int np = __popc(P);
        const double *sw = d.seg + ((size_t)w * L + c2) * L;
        unsigned int bestk = 0xFFFFFFFFu;
        for (int item = tid; item < c2 * np; item += blockDim.x) {
            const int c = item / np, vi = item - c * np;
            const int v = __fns(P, 0, vi + 1);
            const double a = d.table[((size_t)P * k + v) * L + c];
            const double b = d.gam[((size_t)w * k + v) * L + c];
            double mx = a > b ? a : b;
            mx = sw[c] > mx ? sw[c] : mx;
            if (mx <= beta) {
                const unsigned int kk = ((unsigned)c << 5) | (unsigned)v;
                bestk = kk < bestk ? kk : bestk;
            }
        }
        for (int o = 16; o; o >>= 1) {
            const unsigned int other = __shfl_xor_sync(0xFFFFFFFFu, bestk, o);
            bestk = other < bestk ? other : bestk;
        }
        if (lane == 0) s_key[wid] = bestk;
        __syncthreads();
        if (tid == 0) {
            unsigned int x = s_key[0];
            for (int i = 1; i < (int)(blockDim.x >> 5); ++i) x = s_key[i] < x ? s_key[i] : x;
            s_pick = x;
        }
        __syncthreads();
        const unsigned int pick = s_pick;
        if (pick == 0xFFFFFFFFu) {  // cannot happen on a consistent table; report, do not trap
            if (tid == 0) out->status = PP_ERR_CUDA;
            return;
        }
        S = P;
        w = (int)(pick & 31u);
        c2 = (int)(pick >> 5);
        __syncthreads();
    }
}

}  // namespace

cudaError_t launch_compute_search(const CtDev &d, pp_solution *out, cudaStream_t s)
{
    const int k = d.k, L = d.L;
    cudaError_t e = cudaMemsetAsync(d.best_val, 0xFF, 16, s);  // best_val and best_key are adjacent
    if (e != cudaSuccess) return e;
    k_ct_tables<<<k * k + k * L + k, 128, 0, s>>>(d);
    const int top = k < L ? k : L;
    for (int level = 2; level <= top; ++level) {
        unsigned long long n = 1;  // source masks of popcount level - 1
        for (int i = 0; i < level - 1; ++i) n = n * (unsigned)(k - i) / (unsigned)(i + 1);
        const size_t sm = (size_t)(k - (level - 1)) * L * sizeof(double);
        e = cudaFuncSetAttribute(k_ct_level, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        if (e != cudaSuccess) return e;
        k_ct_level<<<(unsigned)n, 128, sm, s>>>(d, level);
    }
    k_ct_best<<<296, 256, 0, s>>>(d, 0);
    k_ct_best<<<296, 256, 0, s>>>(d, 1);
    k_ct_backtrack<<<1, 256, 0, s>>>(d, out);
    return cudaGetLastError();
}

}  // namespace pp
