// Colour-coding k-path search, the inner step of the paper's placement stage (Section 3.2.2:
// the threshold classifier of Eq. 8 and the K-PATH call of Algorithm 2), many queries per launch.
//
// A query keeps the links of the communication graph whose bandwidth is at least its threshold
// (class X of Eq. 8) among the nodes that are still available, and asks for a simple path of kk
// vertices whose vertices carry kk different colours (the colouring is an input: the caller draws
// it), from `start` to `end` when those are given; a walk that reaches `end` early is not continued.
// The table of the colour-coding method, reach[C] = set of vertices at which a colourful path with
// colour set C ends, is a 64-bit vertex mask per colour set and lives in shared memory.  One warp
// per query sweeps the colour sets: a set C hands N(reach[C]), the neighbours of its end vertices,
// to every set C + c, restricted to the vertices of colour c.  The path is rebuilt from the table,
// lowest predecessor first.
#include "pp_internal.cuh"

namespace pp {

namespace {

// One warp per query, lane <-> vertices lane and lane + 32 (n <= 64); the table of a query is the
// warp's slice of shared memory.  The colour sets are taken in numerical order: a set only receives
// from its subsets, which are smaller numbers, so no level structure and no block barrier is needed.
// For a set C the neighbours of reach[C] are the OR of the adjacency masks of its end vertices (each
// lane offers the masks of its two vertices, one warp-wide OR), and lane c hands the neighbours of
// colour c to the set C + c: every lane writes a word of its own.
struct KpathLayout {
    size_t reach, radj, cls, col, total;
};
__host__ __device__ inline KpathLayout kpath_layout(int kk)
{
    KpathLayout l;
    l.reach = 0;
    l.radj = ((size_t)1 << kk) * 8;
    l.cls = l.radj + 64 * 8;
    l.col = l.cls + 16 * 8;
    l.total = l.col + 64;
    return l;
}
__host__ __device__ inline int kpath_warps_per_block(int kk) { return kk <= 9 ? 4 : kk <= 11 ? 2 : 1; }

__device__ __forceinline__ unsigned long long warp_or_u64(unsigned long long x)
{
    const uint32_t lo = __reduce_or_sync(0xFFFFFFFFu, (uint32_t)x);
    const uint32_t hi = __reduce_or_sync(0xFFFFFFFFu, (uint32_t)(x >> 32));
    return ((unsigned long long)hi << 32) | lo;
}

__global__ void __launch_bounds__(128)
k_kpath_colour(int n, int kk, int64_t Q, const uint32_t *__restrict__ bw, const uint32_t *__restrict__ threshold,
               const int32_t *__restrict__ start, const int32_t *__restrict__ end,
               const unsigned long long *__restrict__ alive_q, const uint8_t *__restrict__ colours,
               uint8_t *__restrict__ found, int32_t *__restrict__ path)
{
    extern __shared__ __align__(16) unsigned char smem_kpath[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const KpathLayout lay = kpath_layout(kk);
    unsigned char *base = smem_kpath + (size_t)wid * lay.total;
    unsigned long long *reach = reinterpret_cast<unsigned long long *>(base + lay.reach);  // [2^kk]
    unsigned long long *radj = reinterpret_cast<unsigned long long *>(base + lay.radj);    // [64]
    unsigned long long *cls = reinterpret_cast<unsigned long long *>(base + lay.cls);      // [16]
    uint8_t *col = base + lay.col;                                                         // [64]
    const uint32_t nsets = 1u << kk, full = nsets - 1u;
    for (int64_t q = (int64_t)blockIdx.x * warps + wid; q < Q; q += (int64_t)gridDim.x * warps) {
        const uint32_t t = threshold[q];
        const int s = start[q], u = end[q];
        const unsigned long long alive = alive_q[q] & (n == 64 ? ~0ull : ((1ull << n) - 1ull));
        __syncwarp();
        for (uint32_t C = lane; C < nsets; C += 32) reach[C] = 0ull;
        // adjacency of the class-X subgraph among the available nodes, two vertices per lane
        unsigned long long adj2[2];
        int colv[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int v = lane + 32 * h;
            unsigned long long out = 0ull, in = 0ull;
            if (v < n && ((alive >> v) & 1ull)) {
                for (int w = 0; w < n; ++w) {
                    if (w == v || !((alive >> w) & 1ull)) continue;
                    const uint32_t fwd = bw[v * n + w], back = bw[w * n + v];
                    if (fwd > 0 && fwd >= t) out |= 1ull << w;
                    if (back > 0 && back >= t) in |= 1ull << w;
                }
            }
            adj2[h] = out;
            radj[v] = in;
            colv[h] = v < n ? colours[q * n + v] : 255;
            col[v] = (uint8_t)colv[h];
        }
        // vertices of each colour, and the paths of one vertex
        unsigned long long mine = 0ull;  // lane c: the vertices of colour c
        for (int c = 0; c < kk; ++c) {
            unsigned long long x = 0ull;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int v = lane + 32 * h;
                if (v < n && ((alive >> v) & 1ull) && colv[h] == c) x |= 1ull << v;
            }
            x = warp_or_u64(x);
            if (lane == c) mine = x;
        }
        if (lane < 16) cls[lane] = lane < kk ? mine : 0ull;
        __syncwarp();
        if (lane < kk) {
            unsigned long long first = mine;
            if (s >= 0) first &= (s < 64) ? (1ull << s) : 0ull;
            reach[1u << lane] = first;
        }
        __syncwarp();
        const unsigned long long not_end = (u >= 0 && u < 64) ? ~(1ull << u) : ~0ull;
        const bool my_colour = lane < kk;
        for (uint32_t C = 1; C < full; ++C) {
            const unsigned long long X = reach[C] & not_end;  // a walk that has reached the end vertex stops
            if (!X) continue;
            unsigned long long N = (((X >> lane) & 1ull) ? adj2[0] : 0ull) | (((X >> (lane + 32)) & 1ull) ? adj2[1] : 0ull);
            N = warp_or_u64(N);
            if (my_colour && !((C >> lane) & 1u)) {
                const unsigned long long add = N & mine;
                if (add) reach[C | (1u << lane)] |= add;
            }
            __syncwarp();
        }
        if (lane == 0) {
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

size_t kpath_smem_bytes(int kk) { return kpath_layout(kk).total * kpath_warps_per_block(kk); }

cudaError_t launch_kpath(int n, int kk, int64_t Q, const uint32_t *bw, const uint32_t *threshold, const int32_t *start,
                         const int32_t *end, const unsigned long long *alive, const uint8_t *colours, uint8_t *found,
                         int32_t *path, cudaStream_t s)
{
    if (Q <= 0) return cudaSuccess;
    const size_t sm = kpath_smem_bytes(kk);
    cudaError_t e = cudaFuncSetAttribute(k_kpath_colour, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    const int warps = kpath_warps_per_block(kk);
    int64_t blocks = (Q + warps - 1) / warps;
    const int64_t cap = 148 * 16;
    if (blocks > cap) blocks = cap;
    k_kpath_colour<<<(unsigned)blocks, warps * 32, sm, s>>>(n, kk, Q, bw, threshold, start, end, alive, colours, found,
                                                            path);
    return cudaGetLastError();
}

}  // namespace pp
