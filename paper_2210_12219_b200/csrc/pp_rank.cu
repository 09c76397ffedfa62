// Gamma table (Eq. 3) and its rank compression.
//
// gamma[c][v][w] = bits[c] / bw[v][w] takes at most L*U distinct values, U = number of
// distinct usable bandwidths.  For every distinct bandwidth the L quotients are ascending
// when the layers are visited in ascending order of bits (IEEE division is monotone in the
// numerator), so the rank of a quotient x is 1 + sum over the U sorted lists of the number
// of entries below x.  Equal doubles get equal ranks; the map is strictly increasing.
#include "pp_internal.cuh"

namespace pp {

// One block: order[] = layers sorted by (bits, index), pos[] = inverse permutation.
__global__ void k_order(Dev d)
{
    for (int c = threadIdx.x; c < d.L; c += blockDim.x) {
        uint64_t b = d.bits[c];
        int p = 0;
        for (int o = 0; o < d.L; ++o) {
            uint64_t x = d.bits[o];
            p += (x < b) || (x == b && o < c);
        }
        d.pos[c] = (int16_t)p;
        d.order[p] = (int16_t)c;
    }
}

// gu[u][i]: one correctly rounded fp64 division per entry (never contracted, no fast math).
__global__ void k_quotients(Dev d)
{
    int n = d.U * d.L;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        int u = e / d.L, i = e - u * d.L;
        d.gu[e] = __ddiv_rn((double)d.bits[d.order[i]], (double)d.ubw[u]);
    }
}

// rk[u][i] = 1 + #{(u', i') : gu[u'][i'] < gu[u][i]}.
// Block = one list u (its queries are ascending in i); thread t owns list u' = t, t+blockDim, ...
// and merges it against the block's list held in shared memory, adding its counts with
// shared-memory atomics.  Every step advances one of two cursors, so a merge costs <= 2L steps.
__global__ void k_rank_lists(Dev d)
{
    extern __shared__ unsigned char smem_raw[];
    double *q = reinterpret_cast<double *>(smem_raw);            // [L] this block's list
    unsigned int *cnt = reinterpret_cast<unsigned int *>(q + d.L); // [L]
    const int L = d.L, u = blockIdx.x;
    for (int i = threadIdx.x; i < L; i += blockDim.x) {
        q[i] = d.gu[(size_t)u * L + i];
        cnt[i] = 0;
    }
    __syncthreads();
    for (int u2 = threadIdx.x; u2 < d.U; u2 += blockDim.x) {
        const double *other = d.gu + (size_t)u2 * L;
        int j = 0;  // entries of `other` below the current query
        double oj = other[0];
        for (int i = 0; i < L; ++i) {
            double x = q[i];
            while (j < L && oj < x) {
                ++j;
                if (j < L) oj = other[j];
            }
            if (j) atomicAdd(&cnt[i], (unsigned int)j);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < L; i += blockDim.x) d.rk[(size_t)u * L + i] = 1u + cnt[i];
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
    k_order<<<1, 256, 0, s>>>(d);
    ++*launches;
    if (d.U > 0) {
        int n = d.U * d.L;
        k_quotients<<<(n + 255) / 256, 256, 0, s>>>(d);
        ++*launches;
        size_t sm = (size_t)d.L * (sizeof(double) + sizeof(unsigned int));
        int threads = d.U < 32 ? 32 : (d.U > 256 ? 256 : ((d.U + 31) / 32) * 32);
        k_rank_lists<<<d.U, threads, sm, s>>>(d);
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
