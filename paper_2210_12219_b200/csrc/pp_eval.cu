// Batched beta evaluator: one thread per candidate plan.
// gamma_j = bits[e_j] / bw[n_j][n_{j+1}] (Eq. 3), beta = max_j gamma_j (Eq. 2); validity
// rules as documented in pp.h.  The plan rows are staged through shared memory so that the
// global reads of `ends` and `nodes` are coalesced 128-byte requests.
#include "pp_internal.cuh"

namespace pp {

constexpr int kEvalThreads = 256;

__global__ void __launch_bounds__(kEvalThreads)
k_eval(Dev d, int64_t B, const uint8_t *__restrict__ nseg, const int32_t *__restrict__ ends,
       const int32_t *__restrict__ nodes, double *__restrict__ beta, uint8_t *__restrict__ status)
{
    extern __shared__ int32_t sm[];
    const int k = d.k, L = d.L;
    const int stride = k | 1;  // odd row stride: conflict-free column walks
    int32_t *s_ends = sm;
    int32_t *s_nodes = sm + kEvalThreads * stride;
    const int mmax = k < L ? k : L;
    const double kInf = __longlong_as_double(0x7FF0000000000000ll);

    for (int64_t base = (int64_t)blockIdx.x * kEvalThreads; base < B;
         base += (int64_t)gridDim.x * kEvalThreads) {
        int64_t left = B - base;
        int rows = left < kEvalThreads ? (int)left : kEvalThreads;
        __syncthreads();
        for (int i = threadIdx.x; i < rows * k; i += kEvalThreads) {
            int r = i / k, col = i - r * k;
            s_ends[r * stride + col] = ends[base * k + i];
            s_nodes[r * stride + col] = nodes[base * k + i];
        }
        __syncthreads();
        if (threadIdx.x >= rows) continue;
        const int64_t b = base + threadIdx.x;
        const int32_t *e = s_ends + threadIdx.x * stride;
        const int32_t *n = s_nodes + threadIdx.x * stride;
        const int m = nseg[b];
        int flags = 0;
        double bt = kInf;
        if (m < 1 || m > mmax) {
            flags = PP_PLAN_BAD_NSEG;
        } else {
            uint32_t used = 0;
            for (int j = 0; j < m; ++j) {
                int nj = n[j];
                if (nj < 0 || nj >= k) { flags |= PP_PLAN_BAD_NODE; continue; }
                if ((used >> nj) & 1u) flags |= PP_PLAN_BAD_NODE;
                used |= 1u << nj;
            }
            int prev = -1;
            for (int j = 0; j < m - 1; ++j) {
                int ej = e[j];
                if (ej < 0 || ej > L - 2) flags |= PP_PLAN_BAD_ENDS;
                if (j > 0 && ej <= prev) flags |= PP_PLAN_BAD_ENDS;
                prev = ej;
            }
            if (!flags) {
                double acc = 0.0;
                int first = 0;
                for (int j = 0; j < m; ++j) {
                    int last = (j == m - 1) ? L - 1 : e[j];
                    if (d.M[last + 1] - d.M[first] > d.cap[n[j]]) flags |= PP_PLAN_MEMORY;
                    if (j < m - 1) {
                        uint32_t link = d.bw[n[j] * k + n[j + 1]];
                        if (link == 0) {
                            flags |= PP_PLAN_DEAD_LINK;
                        } else {
                            double g = __ddiv_rn((double)d.bits[last], (double)link);
                            acc = g > acc ? g : acc;
                        }
                    }
                    first = last + 1;
                }
                if (!flags) bt = acc;
            }
        }
        beta[b] = bt;
        status[b] = (uint8_t)flags;
    }
}

// The same scoring for plans in compressed rows: plan b owns the entries [off[b], off[b + 1]) of
// `ends` (16-bit cuts) and `nodes` (8-bit node ids), of which the first nseg[b] - 1 / nseg[b] are
// read.  One thread per plan reads its few dozen bytes straight from global memory: neighbouring
// plans are neighbours in memory, so a warp's loads fall into a handful of cache lines.
__global__ void __launch_bounds__(kEvalThreads)
k_eval_packed(Dev d, int64_t B, int64_t total, const uint8_t *__restrict__ nseg, const uint32_t *__restrict__ off,
              const uint16_t *__restrict__ ends, const uint8_t *__restrict__ nodes, double *__restrict__ beta,
              uint8_t *__restrict__ status)
{
    const int k = d.k, L = d.L;
    const int mmax = k < L ? k : L;
    const double kInf = __longlong_as_double(0x7FF0000000000000ll);
    for (int64_t b = (int64_t)blockIdx.x * kEvalThreads + threadIdx.x; b < B; b += (int64_t)gridDim.x * kEvalThreads) {
        const int m = nseg[b];
        const int64_t o0 = off[b], o1 = off[b + 1];
        int flags = 0;
        double bt = kInf;
        if (m < 1 || m > mmax || o1 < o0 || o1 > total || o1 - o0 < m) {
            flags = PP_PLAN_BAD_NSEG;  // also: a row that does not hold nseg entries
        } else {
            const uint16_t *e = ends + o0;
            const uint8_t *n = nodes + o0;
            uint32_t used = 0;
            int prev = -1, first = 0, nprev = -1;
            double acc = 0.0;
            int mem_dead = 0;
            for (int j = 0; j < m; ++j) {
                const int nj = n[j];
                if (nj >= k) { flags |= PP_PLAN_BAD_NODE; continue; }
                if ((used >> nj) & 1u) flags |= PP_PLAN_BAD_NODE;
                used |= 1u << nj;
            }
            for (int j = 0; j < m - 1; ++j) {
                const int ej = e[j];
                if (ej > L - 2) flags |= PP_PLAN_BAD_ENDS;
                if (j > 0 && ej <= prev) flags |= PP_PLAN_BAD_ENDS;
                prev = ej;
            }
            if (!flags) {
                for (int j = 0; j < m; ++j) {
                    const int last = (j == m - 1) ? L - 1 : e[j];
                    const int nj = n[j];
                    if (d.M[last + 1] - d.M[first] > d.cap[nj]) mem_dead |= PP_PLAN_MEMORY;
                    if (j > 0) {
                        const uint32_t link = d.bw[nprev * k + nj];
                        if (link == 0) {
                            mem_dead |= PP_PLAN_DEAD_LINK;
                        } else {
                            const double g = __ddiv_rn((double)d.bits[first - 1], (double)link);
                            acc = g > acc ? g : acc;
                        }
                    }
                    nprev = nj;
                    first = last + 1;
                }
                flags |= mem_dead;
                if (!flags) bt = acc;
            }
        }
        beta[b] = bt;
        status[b] = (uint8_t)flags;
    }
}

cudaError_t launch_eval_packed(const Dev &d, int64_t B, int64_t total, const uint8_t *nseg, const uint32_t *off,
                               const uint16_t *ends, const uint8_t *nodes, double *beta, uint8_t *status,
                               cudaStream_t s)
{
    if (B <= 0) return cudaSuccess;
    int64_t blocks = (B + kEvalThreads - 1) / kEvalThreads;
    const int64_t cap = 148 * 16;
    if (blocks > cap) blocks = cap;
    k_eval_packed<<<(unsigned)blocks, kEvalThreads, 0, s>>>(d, B, total, nseg, off, ends, nodes, beta, status);
    return cudaGetLastError();
}

cudaError_t launch_eval(const Dev &d, int64_t B, const uint8_t *nseg, const int32_t *ends,
                        const int32_t *nodes, double *beta, uint8_t *status, cudaStream_t s)
{
    if (B <= 0) return cudaSuccess;
    int64_t blocks = (B + kEvalThreads - 1) / kEvalThreads;
    int64_t cap = 148 * 16;
    if (blocks > cap) blocks = cap;
    size_t sm = (size_t)2 * kEvalThreads * (d.k | 1) * sizeof(int32_t);
    k_eval<<<(unsigned)blocks, kEvalThreads, sm, s>>>(d, B, nseg, ends, nodes, beta, status);
    return cudaGetLastError();
}

}  // namespace pp
