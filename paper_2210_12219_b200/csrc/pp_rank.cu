// Gamma table (Eq. 3) and its rank compression.
//
// gamma[c][v][w] = bits[c] / bw[v][w] takes at most L*U distinct values, U = number of
// distinct usable bandwidths.  For every distinct bandwidth the L quotients are ascending
// when the layers are visited in ascending order of bits (IEEE division is monotone in the
// numerator), so the rank of a quotient x is 1 + sum over the U sorted lists of the number
// of entries below x.  Equal doubles get equal ranks; the map is strictly increasing.
#include "pp_internal.cuh"

namespace pp {

// order[] = layers sorted by (bits, index), pos[] = inverse permutation, then
// gu[u][i] = bits[order[i]] / ubw[u], one correctly rounded fp64 division per entry (never
// contracted, no fast math).  Every block works out the order for itself in shared memory (L is at
// most 1024) and takes its share of the U * L quotients; block 0 also writes order[] and pos[].
__global__ void __launch_bounds__(1024) k_order_quotients(Dev d)
{
    extern __shared__ unsigned char smem_raw[];
    uint64_t *raw = reinterpret_cast<uint64_t *>(smem_raw);  // [L] bits by layer
    uint64_t *sorted = raw + d.L;                            // [L] bits ascending
    for (int c = threadIdx.x; c < d.L; c += blockDim.x) raw[c] = d.bits[c];
    __syncthreads();
    for (int c = threadIdx.x; c < d.L; c += blockDim.x) {
        const uint64_t b = raw[c];
        int p = 0;
        for (int o = 0; o < d.L; ++o) {
            const uint64_t x = raw[o];
            p += (x < b) || (x == b && o < c);
        }
        sorted[p] = b;
        if (blockIdx.x == 0) {
            d.pos[c] = (int16_t)p;
            d.order[p] = (int16_t)c;
        }
    }
    __syncthreads();
    const int n = d.U * d.L;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        int u = e / d.L, i = e - u * d.L;
        d.gu[e] = __ddiv_rn((double)sorted[i], (double)d.ubw[u]);
    }
}

// rk[e] = 1 + #{e' : gu[e'] < gu[e]}.  A block owns kRankQueries quotients and streams all U
// lists through shared memory in tiles; thread (q, g) binary-searches the lists g, g+4, ... of
// each tile for query q, and the four partial counts meet in a shared-memory atomic.
constexpr int kRankQueries = 256;
constexpr int kRankGroups = 4;
constexpr int kRankTileBytes = 48 * 1024;

__global__ void __launch_bounds__(kRankQueries *kRankGroups) k_rank(Dev d, int tile_lists)
{
    extern __shared__ unsigned char smem_raw[];
    double *tile = reinterpret_cast<double *>(smem_raw);  // [tile_lists][L]
    __shared__ unsigned int s_cnt[kRankQueries];
    const int L = d.L, U = d.U, n = U * L;
    const int q = threadIdx.x % kRankQueries, grp = threadIdx.x / kRankQueries;
    const int e = blockIdx.x * kRankQueries + q;
    const double x = e < n ? d.gu[e] : 0.0;
    if (grp == 0) s_cnt[q] = 0;
    unsigned int below = 0;
    for (int u0 = 0; u0 < U; u0 += tile_lists) {
        const int nl = (U - u0 < tile_lists) ? U - u0 : tile_lists;
        __syncthreads();
        for (int i = threadIdx.x; i < nl * L; i += blockDim.x) tile[i] = d.gu[(size_t)u0 * L + i];
        __syncthreads();
        if (e < n)
            for (int l = grp; l < nl; l += kRankGroups) {
                const double *list = tile + l * L;
                int a = 0, b = L;  // first index with list[idx] >= x
                while (a < b) {
                    const int mid = (a + b) >> 1;
                    if (list[mid] < x) a = mid + 1; else b = mid;
                }
                below += (unsigned)a;
            }
    }
    if (e < n && below) atomicAdd(&s_cnt[q], below);
    __syncthreads();
    if (grp == 0 && e < n) {
        const unsigned int r = 1u + s_cnt[q];
        d.rk[e] = r;
        d.inv[r] = (uint32_t)e;  // any entry of that rank will do
    }
}

template <typename T>
__global__ void k_expand(Dev d)
{
    const T kInf = (T)~(T)0;
    T *rank = reinterpret_cast<T *>(d.rank);
    int rows = d.k * d.k;
    for (int r = blockIdx.x; r < rows; r += gridDim.x) {
        int w = r / d.k, v = r - w * d.k;
        int u = (v == w) ? -1 : d.pair_u[v * d.k + w];
        for (int c = threadIdx.x; c < d.Lpad; c += blockDim.x) {
            T x = kInf;
            if (u >= 0 && c < d.L) x = (T)d.rk[(size_t)u * d.L + d.pos[c]];
            rank[(size_t)r * d.Lpad + c] = x;
        }
    }
}

cudaError_t launch_rank_build(const Dev &d, cudaStream_t s, int *launches)
{
    *launches = 0;
    {
        const int n = d.U * d.L;
        int blocks = (n + 1023) / 1024;
        if (blocks < 1) blocks = 1;
        if (blocks > 64) blocks = 64;
        k_order_quotients<<<blocks, 1024, 2 * (size_t)d.L * sizeof(uint64_t), s>>>(d);
    }
    ++*launches;
    if (d.U > 0) {
        int tile_lists = kRankTileBytes / (int)(d.L * sizeof(double));
        if (tile_lists < 1) tile_lists = 1;
        if (tile_lists > d.U) tile_lists = d.U;
        const size_t sm = (size_t)tile_lists * d.L * sizeof(double);
        cudaError_t e = cudaFuncSetAttribute(k_rank, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        if (e != cudaSuccess) return e;
        const int n = d.U * d.L;
        k_rank<<<(n + kRankQueries - 1) / kRankQueries, kRankQueries * kRankGroups, sm, s>>>(d, tile_lists);
        ++*launches;
    }
    if (d.elem == 2)
        k_expand<uint16_t><<<d.k * d.k, 128, 0, s>>>(d);
    else
        k_expand<uint32_t><<<d.k * d.k, 128, 0, s>>>(d);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace pp
