// Many-instance exact search: one thread block per instance, the whole state table in shared
// memory.  Same recurrence, final choice and backtrack rule as the single-instance path (see
// pp_sweep.cu), but small enough that values are kept as the gamma doubles themselves:
// fmin/fmax on non-negative doubles only select, so results are bit-identical to the ranked
// path.  Global memory sees the inputs once and the result record once.
#include "pp_internal.cuh"

namespace pp {

constexpr int kBatchThreads = 1024;
constexpr int kBatchWarps = kBatchThreads / 32;

struct BatchLayout {
    size_t dp, gam, gs, M, cap, lo, rowoff, mlist, loff, total;
};

__host__ __device__ inline BatchLayout batch_layout(int L, int k)
{
    BatchLayout b;
    size_t rows = (size_t)k << (k - 1);
    size_t o = 0;
    b.dp = o;      o += rows * L * sizeof(double);
    b.gam = o;     o += (size_t)L * k * k * sizeof(double);
    b.gs = o;      o += (size_t)kBatchWarps * L * sizeof(double);
    b.M = o;       o += (size_t)(L + 1) * sizeof(uint64_t);
    b.cap = o;     o += (size_t)k * sizeof(uint64_t);
    b.rowoff = o;  o += ((size_t)1 << k) * sizeof(uint32_t);
    b.loff = o;    o += (size_t)(k + 2) * sizeof(uint32_t);
    b.mlist = o;   o += ((size_t)1 << k) * sizeof(uint16_t);
    b.lo = o;      o += (size_t)k * L * sizeof(int16_t);
    b.total = (o + 15) & ~(size_t)15;
    return b;
}

size_t batch_smem_bytes(int L, int k)
{
    if (k > 15) return (size_t)1 << 40;
    return batch_layout(L, k).total;
}

// number of set bits in all integers below S
__device__ inline uint32_t bits_below(uint32_t S, int k)
{
    uint32_t t = 0;
    for (int b = 0; b < k; ++b) {
        uint32_t cyc = (S >> (b + 1)) << b;
        uint32_t rem = S & ((2u << b) - 1u);
        t += cyc + (rem > (1u << b) ? rem - (1u << b) : 0u);
    }
    return t;
}

// Work split inside a block: one warp per target row (S', w), lanes over the cut position.  The
// warp first forms g[c] = min_v max(dp[S'\{w}][v][c], gamma[c][v][w]) into its own shared-memory
// strip, then every lane scans its window [lo_w(c'), c'-1] of that strip.  Rows, gamma[v][w][.]
// and the strip are all read with consecutive lanes on consecutive addresses.
__global__ void __launch_bounds__(kBatchThreads, 1)
k_batch(int64_t B, int L, int k, const uint64_t *__restrict__ g_bits,
        const uint64_t *__restrict__ g_mem, const uint64_t *__restrict__ g_cap,
        const uint32_t *__restrict__ g_bw, double *__restrict__ o_beta, int32_t *__restrict__ o_m,
        int32_t *__restrict__ o_cuts, int32_t *__restrict__ o_place, int8_t *__restrict__ o_status)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const BatchLayout lay = batch_layout(L, k);
    double *dp = reinterpret_cast<double *>(smem + lay.dp);
    double *gam = reinterpret_cast<double *>(smem + lay.gam);  // [v][w][c]
    uint64_t *M = reinterpret_cast<uint64_t *>(smem + lay.M);
    uint64_t *cap = reinterpret_cast<uint64_t *>(smem + lay.cap);
    uint32_t *rowoff = reinterpret_cast<uint32_t *>(smem + lay.rowoff);
    uint32_t *loff = reinterpret_cast<uint32_t *>(smem + lay.loff);
    uint16_t *mlist = reinterpret_cast<uint16_t *>(smem + lay.mlist);
    int16_t *lo = reinterpret_cast<int16_t *>(smem + lay.lo);
    __shared__ unsigned long long s_val[kBatchWarps];
    __shared__ unsigned int s_tie[kBatchWarps];
    __shared__ unsigned long long s_bestval;
    __shared__ unsigned int s_besttie;
    __shared__ int s_bad;

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    double *gs = reinterpret_cast<double *>(smem + lay.gs) + (size_t)wid * L;
    const uint32_t nm = 1u << k;
    const double kInf = __longlong_as_double(0x7FF0000000000000ll);
    const unsigned long long kInfBits = 0x7FF0000000000000ull;

    // instance-independent tables
    for (uint32_t S = tid; S < nm; S += kBatchThreads) rowoff[S] = bits_below(S, k);
    if (tid <= k) {  // thread j lists the masks of popcount j
        uint32_t cnt = 0;
        for (uint32_t S = 0; S < nm; ++S) cnt += (__popc(S) < tid);
        loff[tid] = cnt;
        if (tid == k) loff[k + 1] = nm;
    }
    __syncthreads();
    if (tid <= k) {
        uint32_t at = loff[tid];
        for (uint32_t S = 0; S < nm; ++S)
            if (__popc(S) == tid) mlist[at++] = (uint16_t)S;
    }

    for (int64_t inst = blockIdx.x; inst < B; inst += gridDim.x) {
        const uint64_t *bits = g_bits + inst * L;
        const uint64_t *mem = g_mem + inst * L;
        const uint32_t *bw = g_bw + inst * k * k;
        __syncthreads();
        if (tid == 0) {
            s_bad = 0;
            uint64_t acc = 0;
            M[0] = 0;
            for (int i = 0; i < L; ++i) { acc += mem[i]; M[i + 1] = acc; }
        }
        if (tid < k) cap[tid] = g_cap[inst * k + tid];
        __syncthreads();
        for (int e = tid; e < L * k * k; e += kBatchThreads) {
            int r = e / L, c = e - r * L, v = r / k, w = r - v * k;
            uint64_t b = bits[c];
            uint32_t link = bw[r];
            if (b >= PP_MAX_BITS || link >= PP_MAX_KBPS) s_bad = 1;
            gam[e] = (v == w || link == 0) ? kInf : __ddiv_rn((double)b, (double)link);
        }
        // lo[w][c'] = first c >= 0 such that layers c+1..c' fit on w (c' if none)
        for (int e = tid; e < k * L; e += kBatchThreads) {
            int w = e / L, c2 = e - w * L;
            int c = c2;  // step down while the segment starting at layer c (previous cut c-1) fits
            while (c > 0 && M[c2 + 1] - M[c] <= cap[w]) --c;
            lo[e] = (int16_t)c;
        }
        // base frontier
        for (int e = tid; e < k * L; e += kBatchThreads) {
            int v = e / L, c = e - v * L;
            dp[(size_t)rowoff[1u << v] * L + c] = (M[c + 1] <= cap[v]) ? 0.0 : kInf;
        }
        __syncthreads();
        const int bad = s_bad;
        const int jmax = k < L ? k : L;
        for (int j = 2; j <= k; ++j) {
            const uint32_t nrows = (loff[j + 1] - loff[j]) * j;
            for (uint32_t rr = wid; rr < nrows; rr += kBatchWarps) {
                const uint32_t mi = rr / j;
                const int wi = rr - mi * j;
                const uint32_t S2 = mlist[loff[j] + mi];
                uint32_t t = S2;
                for (int i = 0; i < wi; ++i) t &= t - 1;
                const int w = __ffs(t) - 1;
                const uint32_t P = S2 & ~(1u << w);
                double *out = dp + (size_t)(rowoff[S2] + wi) * L;
                if (j > jmax) {
                    for (int c = lane; c < L; c += 32) out[c] = kInf;
                    continue;
                }
                const double *src0 = dp + (size_t)rowoff[P] * L;
                for (int c = lane; c < L; c += 32) {
                    double g = kInf;
                    int vi = 0;
                    for (uint32_t rem = P; rem; rem &= rem - 1, ++vi) {
                        const int v = __ffs(rem) - 1;
                        g = fmin(g, fmax(src0[vi * L + c], gam[(v * k + w) * L + c]));
                    }
                    gs[c] = g;
                }
                __syncwarp();
                for (int c2 = lane; c2 < L; c2 += 32) {
                    double best = kInf;
                    for (int c = lo[w * L + c2]; c < c2; ++c) best = fmin(best, gs[c]);
                    out[c2] = best;
                }
                __syncwarp();
            }
            __syncthreads();
        }
        // final state: lexicographic minimum of (value, popcount, mask, node) at c = L-1
        unsigned long long bv = kInfBits;
        unsigned int bt = 0xFFFFFFFFu;
        for (uint32_t e = tid; e < nm * (uint32_t)k; e += kBatchThreads) {
            uint32_t S = e / k;
            int v = e - S * k;
            if (!((S >> v) & 1u)) continue;
            double x = dp[(size_t)(rowoff[S] + __popc(S & ((1u << v) - 1u))) * L + (L - 1)];
            unsigned long long xb = (unsigned long long)__double_as_longlong(x);
            unsigned int tie = ((unsigned)__popc(S) << 25) | (S << 5) | (unsigned)v;
            if (xb < bv || (xb == bv && tie < bt)) { bv = xb; bt = tie; }
        }
        for (int o = 16; o; o >>= 1) {
            unsigned long long ov = __shfl_xor_sync(0xFFFFFFFFu, bv, o);
            unsigned int ot = __shfl_xor_sync(0xFFFFFFFFu, bt, o);
            if (ov < bv || (ov == bv && ot < bt)) { bv = ov; bt = ot; }
        }
        if (lane == 0) { s_val[wid] = bv; s_tie[wid] = bt; }
        __syncthreads();
        if (tid == 0) {
            for (int i = 1; i < kBatchThreads / 32; ++i)
                if (s_val[i] < bv || (s_val[i] == bv && s_tie[i] < bt)) { bv = s_val[i]; bt = s_tie[i]; }
            s_bestval = bv;
            s_besttie = bt;
        }
        __syncthreads();
        bv = s_bestval;
        bt = s_besttie;
        int32_t *cuts = o_cuts ? o_cuts + inst * (k - 1) : nullptr;
        int32_t *place = o_place + inst * k;
        if (tid < k) place[tid] = -1;
        if (cuts && tid < k - 1) cuts[tid] = -1;
        __syncthreads();
        if (bad || bv >= kInfBits) {
            if (tid == 0) {
                o_beta[inst] = kInf;
                o_m[inst] = 0;
                o_status[inst] = bad ? (int8_t)PP_ERR_LIMIT : (int8_t)PP_INFEASIBLE;
            }
            continue;
        }
        if (wid == 0) {  // backtrack by one warp
            const double bstar = __longlong_as_double((long long)bv);
            const int m = (int)(bt >> 25);
            uint32_t S = (bt >> 5) & 0xFFFFFu;
            int w = (int)(bt & 31u), c2 = L - 1;
            if (lane == 0) {
                o_beta[inst] = bstar;
                o_m[inst] = m;
                o_status[inst] = (int8_t)PP_OK;
            }
            for (int j = m - 1; j >= 0; --j) {
                if (lane == 0) {
                    place[j] = w;
                    if (j < m - 1) cuts[j] = c2;
                }
                if (j == 0) break;
                uint32_t P = S & ~(1u << w);
                int l0 = lo[w * L + c2];
                unsigned int pick = 0xFFFFFFFFu;
                for (int it = lane; it < (c2 - l0) * k; it += 32) {
                    int c = l0 + it / k, v = it - (it / k) * k;
                    if (!((P >> v) & 1u)) continue;
                    double a = dp[(size_t)(rowoff[P] + __popc(P & ((1u << v) - 1u))) * L + c];
                    double cand = fmax(a, gam[(v * k + w) * L + c]);
                    if (cand <= bstar) {
                        unsigned int kk = ((unsigned)c << 5) | (unsigned)v;
                        pick = kk < pick ? kk : pick;
                    }
                }
                for (int o = 16; o; o >>= 1) {
                    unsigned int other = __shfl_xor_sync(0xFFFFFFFFu, pick, o);
                    pick = other < pick ? other : pick;
                }
                if (pick == 0xFFFFFFFFu) {  // inconsistent table: flag the instance, keep going
                    if (lane == 0) o_status[inst] = (int8_t)PP_ERR_CUDA;
                    break;
                }
                S = P;
                w = (int)(pick & 31u);
                c2 = (int)(pick >> 5);
            }
        }
    }
}

cudaError_t launch_batch(int64_t B, int L, int k, const uint64_t *bits, const uint64_t *mem,
                         const uint64_t *cap, const uint32_t *bw, double *beta, int32_t *m,
                         int32_t *cuts, int32_t *placement, int8_t *status, cudaStream_t s)
{
    if (B <= 0) return cudaSuccess;
    size_t sm = batch_smem_bytes(L, k);
    cudaError_t e = cudaFuncSetAttribute(k_batch, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148, per_sm = 1;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_batch, kBatchThreads, sm);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    int64_t grid = (int64_t)sms * per_sm;
    if (grid > B) grid = B;
    k_batch<<<(unsigned)grid, kBatchThreads, sm, s>>>(B, L, k, bits, mem, cap, bw, beta, m, cuts,
                                                      placement, status);
    return cudaGetLastError();
}

}  // namespace pp
