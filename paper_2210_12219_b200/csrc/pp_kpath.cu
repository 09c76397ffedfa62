// Colour-coding k-path search, the inner step of the paper's placement stage (Section 3.2.2:
// the threshold classifier of Eq. 8 and the K-PATH call of Algorithm 2), many queries per launch.
//
// A query keeps the links of the communication graph whose bandwidth is at least its threshold
// (class X of Eq. 8) among the nodes that are still available, and asks for a simple path of kk
// vertices whose vertices carry kk different colours (the colouring is an input: the caller draws
// it), from `start` to `end` when those are given; a walk that reaches `end` early is not continued.
// The table of the colour-coding method, reach[C] = set of vertices at which a colourful path with
// colour set C ends, is a 64-bit vertex mask per colour set and lives in shared memory.  One block
// per query sweeps the colour sets by popcount, like the node sets of the exact search: a set C
// hands N(reach[C]), the neighbours of its end vertices, to every set C + c, restricted to the
// vertices of colour c.  The path is rebuilt from the table, lowest predecessor first.
#include "pp_internal.cuh"

namespace pp {

namespace {

constexpr int kKpathThreads = 128;

__global__ void __launch_bounds__(kKpathThreads)
k_kpath_colour(int n, int kk, int64_t Q, const uint32_t *__restrict__ bw, const uint32_t *__restrict__ threshold,
               const int32_t *__restrict__ start, const int32_t *__restrict__ end,
               const unsigned long long *__restrict__ alive_q, const uint8_t *__restrict__ colours,
               uint8_t *__restrict__ found, int32_t *__restrict__ path)
{
    extern __shared__ unsigned long long reach[];  // [2^kk]
    __shared__ unsigned long long adj[64], radj[64], cls[16];
    __shared__ uint8_t col[64];
    const int tid = threadIdx.x;
    const uint32_t nsets = 1u << kk, full = nsets - 1u;
    for (int64_t q = blockIdx.x; q < Q; q += gridDim.x) {
        const uint32_t t = threshold[q];
        const int s = start[q], u = end[q];
        const unsigned long long alive = alive_q[q] & (n == 64 ? ~0ull : ((1ull << n) - 1ull));
        __syncthreads();
        for (uint32_t C = tid; C < nsets; C += kKpathThreads) reach[C] = 0ull;
        if (tid < 16) cls[tid] = 0ull;
        if (tid < 64) {
            unsigned long long out = 0ull, in = 0ull;
            if (tid < n && ((alive >> tid) & 1ull)) {
                for (int w = 0; w < n; ++w) {
                    if (w == tid || !((alive >> w) & 1ull)) continue;
                    const uint32_t fwd = bw[tid * n + w], back = bw[w * n + tid];
                    if (fwd > 0 && fwd >= t) out |= 1ull << w;
                    if (back > 0 && back >= t) in |= 1ull << w;
                }
            }
            adj[tid] = out;
            radj[tid] = in;
            col[tid] = tid < n ? colours[q * n + tid] : (uint8_t)255;
        }
        __syncthreads();
        if (tid < n && ((alive >> tid) & 1ull) && col[tid] < kk) {
            atomicOr(&cls[col[tid]], 1ull << tid);                                           // vertices of each colour
            if (s < 0 || s == tid) atomicOr(&reach[1u << col[tid]], 1ull << tid);  // paths of one vertex
        }
        __syncthreads();
        const unsigned long long not_end = (u >= 0 && u < 64) ? ~(1ull << u) : ~0ull;
        for (int level = 1; level < kk; ++level) {
            for (uint32_t C = 1 + tid; C < nsets; C += kKpathThreads) {
                if (__popc(C) != level) continue;
                unsigned long long X = reach[C] & not_end;  // a walk that has reached the end vertex stops
                if (!X) continue;
                unsigned long long N = 0ull;
                while (X) {
                    const int v = __ffsll((long long)X) - 1;
                    X &= X - 1ull;
                    N |= adj[v];
                }
                for (uint32_t rem = full & ~C; rem; rem &= rem - 1u) {
                    const int c = __ffs(rem) - 1;
                    const unsigned long long add = N & cls[c];
                    if (add) atomicOr(&reach[C | (1u << c)], add);
                }
            }
            __syncthreads();
        }
        if (tid == 0) {
            unsigned long long ends = reach[full];
            if (u >= 0) ends &= (u < 64) ? (1ull << u) : 0ull;
            int32_t *out = path + q * kk;
            if (!ends) {
                found[q] = 0;
                for (int i = 0; i < kk; ++i) out[i] = -1;
            } else {
                found[q] = 1;
                int v = __ffsll((long long)ends) - 1;
                uint32_t C = full;
                out[kk - 1] = v;
                for (int i = kk - 2; i >= 0; --i) {
                    C &= ~(1u << col[v]);
                    const unsigned long long cand = reach[C] & radj[v] & not_end;
                    v = __ffsll((long long)cand) - 1;  // never empty: v was reached from such a vertex
                    out[i] = v;
                }
            }
        }
    }
}

}  // namespace

size_t kpath_smem_bytes(int kk) { return ((size_t)1 << kk) * sizeof(unsigned long long); }

cudaError_t launch_kpath(int n, int kk, int64_t Q, const uint32_t *bw, const uint32_t *threshold, const int32_t *start,
                         const int32_t *end, const unsigned long long *alive, const uint8_t *colours, uint8_t *found,
                         int32_t *path, cudaStream_t s)
{
    if (Q <= 0) return cudaSuccess;
    const size_t sm = kpath_smem_bytes(kk);
    cudaError_t e = cudaFuncSetAttribute(k_kpath_colour, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    int64_t blocks = Q;
    const int64_t cap = 148 * 16;
    if (blocks > cap) blocks = cap;
    k_kpath_colour<<<(unsigned)blocks, kKpathThreads, sm, s>>>(n, kk, Q, bw, threshold, start, end, alive, colours,
                                                                found, path);
    return cudaGetLastError();
}

}  // namespace pp
