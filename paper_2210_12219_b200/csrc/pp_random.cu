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

constexpr int kRandomThreads = 128;

// Rows travel through shared memory so that global memory sees whole contiguous blocks: the draws
// of the block's plans on the way in, their two output rows on the way out.  A thread's outputs
// overwrite its own draws: step s has read words 2s and 2s+1 before segment n <= s + 1 goes to
// words 2(n-1) (cut) and 2(n-1)+1 (node).  The row stride is odd, which keeps the threads of a
// warp, each on its own row, on different banks.  The prefix sums and capacities are staged too:
// the bisection reads them at dependent addresses.
__global__ void __launch_bounds__(kRandomThreads)
k_random_plans(Dev d, int64_t P, const uint32_t *__restrict__ draws, uint8_t *nseg, int32_t *ends, int32_t *nodes)
{
    extern __shared__ uint32_t smem_words[];
    const int k = d.k, L = d.L, W = 2 * k, stride = W + 1, tid = threadIdx.x;
    uint32_t *sd = smem_words;  // [threads][stride]: draws in, (cut, node) pairs out
    uint64_t *sM = reinterpret_cast<uint64_t *>(smem_words + ((kRandomThreads * stride + 1) & ~1));  // [L+1]
    uint64_t *scap = sM + L + 1;                                                                     // [k]
    for (int i = tid; i <= L; i += kRandomThreads) sM[i] = d.M[i];
    for (int i = tid; i < k; i += kRandomThreads) scap[i] = d.cap[i];
    const int64_t p0 = (int64_t)blockIdx.x * kRandomThreads;
    const int np = P - p0 < kRandomThreads ? (int)(P - p0) : kRandomThreads;
    {
        const uint32_t *src = draws + p0 * W;
        int r = tid / W, c = tid - r * W;
        const int dr = kRandomThreads / W, dc = kRandomThreads - dr * W;
        for (int i = tid; i < np * W; i += kRandomThreads) {
            sd[r * stride + c] = src[i];
            r += dr;
            c += dc;
            if (c >= W) { c -= W; ++r; }
        }
    }
    __syncthreads();
    if (tid < np) {
        const uint32_t *dr = sd + tid * stride;
        int32_t *out = reinterpret_cast<int32_t *>(sd + tid * stride);
        uint32_t used = 0;
        int first = 0, n = 0;
        bool done = false;
        for (int step = 0; step < k; ++step) {
            // node: the r-th node not used yet
            int r = (int)(((unsigned long long)dr[2 * step] * (unsigned)(k - step)) >> 32);
            uint32_t free_nodes = ~used & ((1u << k) - 1u);
            for (; r > 0; --r) free_nodes &= free_nodes - 1;
            const int node = __ffs(free_nodes) - 1;
            // segments [first, e] that fit: prefix sums ascend, so a bisection finds how many
            const uint64_t base = sM[first], room = scap[node];
            int lo = first, hi = L;  // every e < lo fits, no e >= hi does
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (sM[mid + 1] - base <= room) lo = mid + 1; else hi = mid;
            }
            const int count = lo - first;
            if (count == 0) break;
            const int last = first + (int)(((unsigned long long)dr[2 * step + 1] * (unsigned)count) >> 32);
            used |= 1u << node;
            out[2 * n + 1] = node;
            ++n;
            if (last == L - 1) {
                done = true;
                break;
            }
            out[2 * n - 2] = last;
            first = last + 1;
        }
        if (!done) n = 0;
        nseg[p0 + tid] = (uint8_t)n;
        for (int i = n; i < k; ++i) out[2 * i + 1] = -1;
        for (int i = n > 0 ? n - 1 : 0; i < k; ++i) out[2 * i] = -1;
    }
    __syncthreads();
    {
        int32_t *de = ends + p0 * k, *dn = nodes + p0 * k;
        int r = tid / k, c = tid - r * k;
        const int dr = kRandomThreads / k, dc = kRandomThreads - dr * k;
        for (int i = tid; i < np * k; i += kRandomThreads) {
            de[i] = (int32_t)sd[r * stride + 2 * c];
            dn[i] = (int32_t)sd[r * stride + 2 * c + 1];
            r += dr;
            c += dc;
            if (c >= k) { c -= k; ++r; }
        }
    }
}

cudaError_t launch_random_plans(const Dev &d, int64_t P, const uint32_t *draws, uint8_t *nseg, int32_t *ends,
                                int32_t *nodes, cudaStream_t s)
{
    const int64_t blocks = (P + kRandomThreads - 1) / kRandomThreads;
    if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
    const size_t smem = (((size_t)kRandomThreads * (2 * d.k + 1) + 1) & ~(size_t)1) * sizeof(uint32_t) +
                        ((size_t)d.L + 1 + d.k) * sizeof(uint64_t);  // at most 29 KB (k = 20, L = 1024)
    k_random_plans<<<(unsigned)blocks, kRandomThreads, smem, s>>>(d, P, draws, nseg, ends, nodes);
    return cudaGetLastError();
}

}  // namespace pp
