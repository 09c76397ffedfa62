// Greedy comparison baseline of Section 4 (the "joint-optimization" algorithm of the paper's
// comparison list), many instances per launch: a group of G lanes per instance (G = k rounded up
// to a power of two, so a warp holds 32 / G instances), lane n of the group walks from start node n.
//
// A walk alternates two choices until the chain is used up.  Segment choice: on the current node,
// among the segments that start at the next unassigned layer and fit the node's memory, the one
// whose outgoing transfer is smallest.  Next-node choice: the unused node behind the current
// node's fastest outgoing link.  The result is the walk with the smallest bottleneck latency over
// all start nodes (Eq. 2 with one correctly rounded fp64 division per cut, Eq. 3).  Where the
// paper is silent: a segment that reaches the last layer transfers nothing and is taken as soon
// as it fits; equal transfers take the longer segment, equal links the lower node, equal
// bottlenecks the lower start node; a link of bandwidth 0 is no link; a walk that gets stuck
// contributes no plan.
//
// The work of an instance is a few hundred dependent scalar steps per walk, data-dependent in
// length: with enough instances in flight the kernel is bound by instruction issue (scalar integer
// work on the ALU pipe), far from any bandwidth.
#include "pp_internal.cuh"

namespace pp {

constexpr int kGreedyWarps = 4;

__global__ void __launch_bounds__(kGreedyWarps * 32)
k_greedy_batch(int64_t B, int L, int k, int group, const uint64_t *__restrict__ bits, const uint64_t *__restrict__ mem,
               const uint64_t *__restrict__ cap, const uint32_t *__restrict__ bw, double *o_beta,
               int32_t *o_m, int32_t *o_cuts, int32_t *o_place, int8_t *o_status)
{
    const int per_warp = 32 / group;
    const int lane = threadIdx.x & (group - 1);  // position inside the instance's group = start node
    const int64_t warp = (int64_t)blockIdx.x * kGreedyWarps + (threadIdx.x >> 5);
    int64_t inst = warp * per_warp + (threadIdx.x & 31) / group;
    const bool live = inst < B;  // lanes past the end stay for the shuffles and write nothing
    if (!live) inst = B - 1;
    const uint64_t *b = bits + inst * L, *mm = mem + inst * L, *cp = cap + inst * k;
    const uint32_t *links = bw + inst * k * k;
    int cuts[PP_MAX_K], nodes[PP_MAX_K];
    int nseg = 0;
    double beta = 0.0;
    bool arrived = false;
    if (live && lane < k) {
        uint32_t used = 1u << lane;
        int node = lane, first = 0;
        nodes[0] = lane;
        nseg = 1;
        for (;;) {
            // segment choice; held never exceeds the capacity, so the sum cannot wrap
            const uint64_t room = cp[node];
            uint64_t held = 0, transfer = 0;
            int chosen = -1;
            for (int e = first; e < L; ++e) {
                const uint64_t need = mm[e];
                if (need > room - held) break;
                held += need;
                const uint64_t x = b[e];
                if (e == L - 1 || chosen < 0 || x <= transfer) {
                    chosen = e;
                    transfer = x;
                }
            }
            if (chosen < 0) break;
            if (chosen == L - 1) {
                arrived = true;
                break;
            }
            // next-node choice; strictly faster links only: the lowest node wins a tie, a zero link never wins
            int next = -1;
            uint32_t fastest = 0;
            for (int w = 0; w < k; ++w) {
                const uint32_t x = links[node * k + w];
                if (!((used >> w) & 1u) && x > fastest) {
                    next = w;
                    fastest = x;
                }
            }
            if (next < 0) break;
            const double g = __ddiv_rn((double)transfer, (double)fastest);
            beta = g > beta ? g : beta;
            cuts[nseg - 1] = chosen;
            nodes[nseg] = next;
            ++nseg;
            used |= 1u << next;
            node = next;
            first = chosen + 1;
        }
    }
    // best walk: smallest (beta, start node); beta >= +0.0, so its bit pattern orders like the value
    unsigned long long key = arrived ? (unsigned long long)__double_as_longlong(beta) : ~0ull;
    int who = lane;
    for (int o = group >> 1; o; o >>= 1) {
        const unsigned long long okey = __shfl_xor_sync(0xFFFFFFFFu, key, o);
        const int owho = __shfl_xor_sync(0xFFFFFFFFu, who, o);
        if (okey < key || (okey == key && owho < who)) {
            key = okey;
            who = owho;
        }
    }
    int32_t *oc = o_cuts ? o_cuts + inst * (k - 1) : nullptr;
    int32_t *op = o_place + inst * k;
    if (!live) return;
    if (key == ~0ull) {
        if (lane == 0) {
            o_beta[inst] = __longlong_as_double(0x7FF0000000000000ll);
            o_m[inst] = 0;
            o_status[inst] = (int8_t)PP_INFEASIBLE;
        }
        if (lane < k) op[lane] = -1;
        if (oc && lane < k - 1) oc[lane] = -1;
        return;
    }
    if (lane == who) {
        o_beta[inst] = beta;
        o_m[inst] = nseg;
        o_status[inst] = (int8_t)PP_OK;
        for (int i = 0; i < k; ++i) op[i] = i < nseg ? nodes[i] : -1;
        if (oc)
            for (int i = 0; i < k - 1; ++i) oc[i] = i < nseg - 1 ? cuts[i] : -1;
    }
}

cudaError_t launch_greedy(int64_t B, int L, int k, const uint64_t *bits, const uint64_t *mem,
                          const uint64_t *cap, const uint32_t *bw, double *beta, int32_t *m, int32_t *cuts,
                          int32_t *place, int8_t *status, cudaStream_t s)
{
    int group = 1;
    while (group < k) group <<= 1;
    const int64_t per_block = (int64_t)kGreedyWarps * (32 / group);
    const int64_t blocks = (B + per_block - 1) / per_block;
    if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
    k_greedy_batch<<<(unsigned)blocks, kGreedyWarps * 32, 0, s>>>(B, L, k, group, bits, mem, cap, bw, beta, m, cuts,
                                                                  place, status);
    return cudaGetLastError();
}

}  // namespace pp
