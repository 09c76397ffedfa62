// Gamma table (Eq. 3), its rank compression, and the base frontier.
//
// gamma[c][v][w] = bits[c] / bw[v][w] takes at most L*U distinct values, U = number of
// distinct usable bandwidths.  For every distinct bandwidth the L quotients are ascending
// when the layers are visited in ascending order of bits (IEEE division is monotone in the
// numerator), so the rank of a quotient x is 1 + sum over the U sorted lists of the number
// of entries below x.  Equal doubles get equal ranks; the map is strictly increasing.
//
// Three launches, chained by programmatic dependent launch (each waits for its predecessor to
// complete before it touches anything, only the launch latency overlaps):
//   k_quotients   layers ordered by bits, one division per (distinct bandwidth, layer); clears the
//                 counters of this solve (per-quotient counts, best final key)
//   k_rank_count  block (q, t) counts, for 256 quotients, the entries below each of them in the t-th
//                 tile of lists (binary searches in shared memory) and adds them up in global memory
//   k_expand_base rank = 1 + count, spread out as rank[w][v][c]; base frontier rows (|S| = 1)
#include "pp_internal.cuh"

namespace pp {

namespace {

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;"); }

// order[] = layers sorted by (bits, index), pos[] = inverse permutation, then
// gu[u][i] = bits[order[i]] / ubw[u], one correctly rounded fp64 division per entry (never
// contracted, no fast math).  Every block works out the order for itself in shared memory (L is at
// most 1024) and takes its share of the U * L quotients; block 0 also writes order[] and pos[].
__global__ void __launch_bounds__(1024) k_quotients(Dev d)
{
    extern __shared__ unsigned char smem_raw[];
    uint64_t *raw = reinterpret_cast<uint64_t *>(smem_raw);  // [L] bits by layer
    uint64_t *sorted = raw + d.L;                            // [L] bits ascending
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsize = gridDim.x * blockDim.x;
    if (gtid == 0) *d.best = kNoBest;
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
    pdl_trigger();
    const int n = d.U * d.L;
    for (int e = gtid; e < n; e += gsize) {
        int u = e / d.L, i = e - u * d.L;
        d.gu[e] = __ddiv_rn((double)sorted[i], (double)d.ubw[u]);
        d.cnt[e] = 0;
    }
}

constexpr int kRankQueries = 256;
constexpr int kRankGroups = 4;
constexpr int kRankTileBytes = 48 * 1024;

// cnt[e] += #{e' in the lists of tile blockIdx.y : gu[e'] < gu[e]} for the 256 quotients of chunk
// blockIdx.x.  Thread (q, g) binary-searches the lists g, g + 4, ... of the tile for query q; the
// four partial counts meet in a shared-memory atomic, one global atomic per query and tile.
__global__ void __launch_bounds__(kRankQueries *kRankGroups) k_rank_count(Dev d, int tile_lists)
{
    extern __shared__ unsigned char smem_raw[];
    double *tile = reinterpret_cast<double *>(smem_raw);  // [nl][L]
    __shared__ unsigned int s_cnt[kRankQueries];
    pdl_wait();
    pdl_trigger();
    const int L = d.L, U = d.U, n = U * L;
    const int q = threadIdx.x % kRankQueries, grp = threadIdx.x / kRankQueries;
    const int e = blockIdx.x * kRankQueries + q;
    const int u0 = blockIdx.y * tile_lists;
    const int nl = (U - u0 < tile_lists) ? U - u0 : tile_lists;
    const double x = e < n ? d.gu[e] : 0.0;
    if (grp == 0) s_cnt[q] = 0;
    for (int i = threadIdx.x; i < nl * L; i += blockDim.x) tile[i] = d.gu[(size_t)u0 * L + i];
    __syncthreads();
    unsigned int below = 0;
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
    if (e < n && below) atomicAdd(&s_cnt[q], below);
    __syncthreads();
    if (grp == 0 && e < n && s_cnt[q]) atomicAdd(&d.cnt[e], s_cnt[q]);
}

// Blocks 0 .. k*k-1: row (w, v) of the rank table, rank[w][v][c] = 1 + cnt of gamma[c][v][w]
// (+inf for a missing link, the diagonal and the pad).  Blocks k*k .. k*k+k-1: the base frontier,
// dp[{v}][v][c] = 0 if layers 0..c fit on v, else +inf (a first segment has no incoming transfer,
// Eq. 2), offered as final state when it reaches the last layer.
// All blocks share the per-quotient ranks rk[] and one witness entry per rank, inv[].
template <typename T>
__global__ void __launch_bounds__(128) k_expand_base(Dev d)
{
    pdl_wait();
    const T kInf = (T)~(T)0;
    const int k = d.k, L = d.L, Lpad = d.Lpad;
    const int n = d.U * L;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const uint32_t r = 1u + d.cnt[e];
        d.rk[e] = r;
        d.inv[r] = (uint32_t)e;  // any entry of that rank will do: equal ranks hold equal doubles
    }
    const int rows = k * k;
    if ((int)blockIdx.x < rows) {
        const int r = blockIdx.x;
        const int w = r / k, v = r - w * k;
        const int u = (v == w) ? -1 : d.pair_u[v * k + w];
        T *rank = reinterpret_cast<T *>(d.rank);
        for (int c = threadIdx.x; c < Lpad; c += blockDim.x) {
            T x = kInf;
            if (u >= 0 && c < L) x = (T)(1u + d.cnt[(size_t)u * L + d.pos[c]]);
            if (PP_IN_BOUNDS(d, (size_t)r * Lpad + c, d.rank_elems)) rank[(size_t)r * Lpad + c] = x;
        }
    } else {
        const int v = blockIdx.x - rows;
        const uint32_t S = 1u << v;
        T *row = reinterpret_cast<T *>(d.table) + ((size_t)S * k + v) * Lpad;
        const uint64_t cap = d.cap[v];
        for (int c = threadIdx.x; c < Lpad; c += blockDim.x) {
            const T x = (c < L && d.M[c + 1] <= cap) ? (T)0 : kInf;
            if (PP_IN_BOUNDS(d, ((size_t)S * k + v) * Lpad + c, d.table_elems)) row[c] = x;
            if (c == L - 1 && x != kInf) atomicMin(d.best, pack_best(0u, 1, S, v));
        }
    }
}

}  // namespace

static cudaError_t launch_after(void (*kernel)(Dev), dim3 grid, dim3 block, size_t smem, cudaStream_t s, const Dev &d)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, d);
}

// Queues the three kernels; *launches receives their number.  After them the rank table, the
// per-quotient ranks, the base frontier and the cleared counters of this solve are in place.
cudaError_t launch_rank_base(const Dev &d, cudaStream_t s, int *launches)
{
    *launches = 0;
    const int n = d.U * d.L;
    {
        int blocks = (n + 1023) / 1024;
        if (blocks < 1) blocks = 1;
        if (blocks > 64) blocks = 64;
        k_quotients<<<blocks, 1024, 2 * (size_t)d.L * sizeof(uint64_t), s>>>(d);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    if (d.U > 0) {
        int tile_lists = kRankTileBytes / (int)(d.L * sizeof(double));
        if (tile_lists < 1) tile_lists = 1;
        if (tile_lists > d.U) tile_lists = d.U;
        const size_t sm = (size_t)tile_lists * d.L * sizeof(double);
        cudaError_t e = cudaFuncSetAttribute(k_rank_count, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((n + kRankQueries - 1) / kRankQueries, (d.U + tile_lists - 1) / tile_lists);
        cfg.blockDim = dim3(kRankQueries * kRankGroups);
        cfg.dynamicSmemBytes = sm;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, k_rank_count, d, tile_lists);
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    cudaError_t e = launch_after(d.elem == 2 ? k_expand_base<uint16_t> : k_expand_base<uint32_t>,
                                 dim3(d.k * d.k + d.k), dim3(128), 0, s, d);
    if (e != cudaSuccess) return e;
    ++*launches;
    return cudaSuccess;
}

}  // namespace pp
