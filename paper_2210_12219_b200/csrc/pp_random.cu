// Random comparison baseline of Section 4 (the "random algorithm" of the paper's comparison list),
// many plans per launch for one problem: one thread per plan.  Step s of a plan takes a random
// node among the nodes not used yet (draw 2 s) and a random segment among those that start at
// the next unassigned layer and fit the node's memory (draw 2 s + 1), until the chain is used up.
// The 32-bit draws are inputs; draw d picks index floor(d * n / 2^32) among n candidates in
// ascending order.  Bandwidths play no part: the plans go to the evaluator afterwards.  No plan
// (nseg = 0, rows of -1) when the chosen node holds not even the next layer, or when all k
// nodes are used and layers are left over.
//
// A plan is 2 k dependent steps of a few dozen scalar instructions; the kernel reads 8 k bytes
// of draws and writes 1 + 8 k bytes per plan, so with enough plans it is bound by HBM bandwidth.
#include "pp_internal.cuh"

namespace pp {

__global__ void __launch_bounds__(256)
k_random_plans(Dev d, int64_t P, const uint32_t *__restrict__ draws, uint8_t *nseg, int32_t *ends, int32_t *nodes)
{
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    const int k = d.k, L = d.L;
    const uint32_t *dr = draws + p * 2 * k;
    int32_t *er = ends + p * k, *nr = nodes + p * k;
    uint32_t used = 0;
    int first = 0, n = 0;
    bool done = false;
    for (int step = 0; step < k; ++step) {
        // node: the r-th node not used yet
        int r = (int)(((unsigned long long)dr[2 * step] * (unsigned)(k - step)) >> 32);
        uint32_t free_nodes = ~used & ((1u << k) - 1u);
        for (; r > 0; --r) free_nodes &= free_nodes - 1;
        const int node = __ffs(free_nodes) - 1;
        // segments [first, e] that fit: e = first .. last_fit (prefix sums ascend, so a bisection finds it)
        const uint64_t base = d.M[first], room = d.cap[node];
        int lo = first, hi = L;  // lo = number of leading layers known to fit + first, hi = first that may not
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (d.M[mid + 1] - base <= room) lo = mid + 1; else hi = mid;
        }
        const int count = lo - first;
        if (count == 0) break;
        const int last = first + (int)(((unsigned long long)dr[2 * step + 1] * (unsigned)count) >> 32);
        used |= 1u << node;
        nr[n++] = node;
        if (last == L - 1) {
            done = true;
            break;
        }
        er[n - 1] = last;
        first = last + 1;
    }
    if (!done) n = 0;
    nseg[p] = (uint8_t)n;
    for (int i = n; i < k; ++i) nr[i] = -1;
    for (int i = n > 0 ? n - 1 : 0; i < k; ++i) er[i] = -1;
}

cudaError_t launch_random_plans(const Dev &d, int64_t P, const uint32_t *draws, uint8_t *nseg, int32_t *ends,
                                int32_t *nodes, cudaStream_t s)
{
    const int64_t blocks = (P + 255) / 256;
    if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
    k_random_plans<<<(unsigned)blocks, 256, 0, s>>>(d, P, draws, nseg, ends, nodes);
    return cudaGetLastError();
}

}  // namespace pp
