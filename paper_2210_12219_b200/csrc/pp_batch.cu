// Many-instance exact search: one thread block per instance, the whole state table in shared
// memory as 16-bit ranks (the quotient matrix and the per-entry ranks of the ranking live in the same bytes
// before the table is written).  Same recurrence, final choice and backtrack rule as the
// single-instance path (see pp_sweep.cu); global memory sees the inputs once and the result
// record once.
//
// Per instance the block
//   1. stages the inputs, builds the memory prefix sums and the window table lo[w][c'];
//   2. rank-compresses gamma (Eq. 3): layers sorted by bits, distinct bandwidths listed, one fp64
//      division per (distinct bandwidth, layer), rank = 1 + number of quotients below, counted by a
//      staircase walk over the matrix of quotients, which ascends along rows and columns;
//   3. sweeps the popcount levels with a flat thread <-> (target row, position) mapping:
//      phase A forms g[c] = min_v max(dp[S'\{w}][v][c], rank[v][w][c]) for every row of the level,
//      two neighbouring positions per thread as one packed u16x2 word, thread <-> (source mask,
//      word) with the source words in registers for all target nodes,
//      phase B takes the window minimum over [lo_w(c'), c'-1];
//   4. reduces the final states to the smallest (value, popcount, mask, node), walks back with
//      the threshold rule, and maps the winning rank back to its quotient.
#include "pp_internal.cuh"

namespace pp {

// Three blocks of 384 threads per SM (at k = 8, L = 24: 73 KB of shared memory and at most 56
// registers per thread): the phases of an instance are short and separated by block barriers, so
// what keeps an SM busy is the number of instances in flight on it.
constexpr int kBatchThreads = 384;
constexpr int kBatchBlocksPerSm = 3;
constexpr int kBatchWarps = kBatchThreads / 32;
constexpr uint16_t kInf16 = 0xFFFFu;

struct BatchLayout {
    size_t dp, g, rank, rk, cnt, skey, M, cap, bits, sbits, bw, ubw, uord, pair_u, pos, lo, rowoff, loff, rowinfo, mlist, moff, total;
};

__host__ __device__ inline BatchLayout batch_layout(int L, int k)
{
    BatchLayout b;
    const size_t rows = (size_t)k << (k - 1);
    // widest level: max_j C(k, j) * j
    size_t best = 0, binom = 1;
    for (int j = 1; j <= k; ++j) {
        binom = binom * (size_t)(k - j + 1) / (size_t)j;
        if (binom * j > best) best = binom * j;
    }
    const size_t U = (size_t)k * (k - 1) > 0 ? (size_t)k * (k - 1) : 1;
    const size_t Ls = ((size_t)L + 1) & ~(size_t)1;  // row stride of the 16-bit tables: even, so that
                                                     // two neighbouring cut positions form one word
    size_t o = 0;
    auto take = [&o](size_t bytes) { size_t at = o; o = (o + bytes + 15) & ~(size_t)15; return at; };
    b.M = take((size_t)(L + 1) * sizeof(uint64_t));
    b.cap = take((size_t)k * sizeof(uint64_t));
    b.bits = take((size_t)L * sizeof(uint64_t));
    b.sbits = take((size_t)L * sizeof(uint64_t));
    b.bw = take((size_t)k * k * sizeof(uint32_t));
    b.ubw = take(U * sizeof(uint32_t));
    b.uord = take(U * sizeof(int16_t));
    b.rowoff = take(((size_t)1 << k) * sizeof(uint32_t));
    b.loff = take((size_t)(k + 2) * sizeof(uint32_t));
    b.rowinfo = take(rows * sizeof(uint32_t));
    b.mlist = take(((size_t)1 << k) * sizeof(uint16_t));
    b.moff = take((size_t)(k + 2) * sizeof(uint32_t));
    // The quotient matrix and the per-entry ranks are dead before the first state is written: they
    // share the bytes of the state table.
    {
        auto up16 = [](size_t x) { return (x + 15) & ~(size_t)15; };
        const size_t keys = ((U + 1) * L + 1) * sizeof(unsigned long long);  // a row of +inf and a pad in front
        const size_t scratch = up16(keys) + up16(U * L * sizeof(uint16_t)) + up16(U * L * sizeof(uint32_t));
        const size_t table = rows * Ls * sizeof(uint16_t);
        b.dp = take(table > scratch ? table : scratch);
        size_t q = b.dp;
        b.skey = q; q += up16(keys);
        b.rk = q;   q += up16(U * L * sizeof(uint16_t));
        b.cnt = q;
    }
    b.g = take(best * Ls * sizeof(uint16_t));
    b.rank = take((size_t)k * k * Ls * sizeof(uint16_t));
    b.pair_u = take((size_t)k * k * sizeof(int16_t));
    b.pos = take((size_t)L * sizeof(int16_t));
    b.lo = take((size_t)k * Ls * sizeof(int16_t));  // row stride Ls: two window starts per 32-bit word
    b.total = o;
    return b;
}

size_t batch_smem_bytes(int L, int k)
{
    if (k > 12) return (size_t)1 << 40;  // row descriptors hold the mask in 12 bits
    if ((size_t)k * (k - 1) * L + 1 > 65534) return (size_t)1 << 40;  // ranks must fit 16 bits
    return batch_layout(L, k).total;
}

// row descriptor: source mask (12 bits) | target node (4 bits) << 12 | compact row of the first
// source row << 16 (the output row is the descriptor's own index)
__device__ __forceinline__ uint32_t info_pack(uint32_t P, int w, uint32_t src0)
{
    return P | ((uint32_t)w << 12) | (src0 << 16);
}

// Phase A of one level for the sources masks of NV nodes: g[(P + w, w)][c] = min over v in P of
// max(dp[P][v][c], rank[v][w][c]) for every node w outside P, two positions per 32-bit word.
struct BatchRelaxArgs {
    const uint16_t *dp;       // [compact row][Ls]
    uint16_t *gbuf;           // [row within the target level][Ls]
    const uint16_t *rank;     // [v][w][Ls]
    const uint32_t *rowoff;   // compact row of (S, lowest node of S)
    const uint16_t *masks;    // the source masks of this level
    uint32_t nmasks;
    uint32_t row0;            // first compact row of the target level
    int k, Lh;
};

template <int NV>
__device__ __forceinline__ void batch_relax(const BatchRelaxArgs &a, int tid)
{
    const int Lh = a.Lh, k = a.k;
    const uint32_t *dp32 = reinterpret_cast<const uint32_t *>(a.dp);
    const uint32_t *rank32 = reinterpret_cast<const uint32_t *>(a.rank);
    uint32_t *g32 = reinterpret_cast<uint32_t *>(a.gbuf);
    const uint32_t items = a.nmasks * (uint32_t)Lh;
    const uint32_t full = (1u << k) - 1u;
    for (uint32_t it = tid; it < items; it += kBatchThreads) {
        const uint32_t pi = it / (uint32_t)Lh;
        const int cw = (int)(it - pi * (uint32_t)Lh);
        const uint32_t P = a.masks[pi];
        const uint32_t *src = dp32 + (size_t)a.rowoff[P] * Lh + cw;
        uint32_t d[NV];
        int roff[NV];  // word offset of rank[v][0][cw]
        uint32_t rem = P;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int v = __ffs(rem) - 1;
            rem &= rem - 1;
            d[i] = src[i * Lh];
            roff[i] = v * k * Lh + cw;
        }
        for (uint32_t wrem = full & ~P; wrem; wrem &= wrem - 1) {
            const int w = __ffs(wrem) - 1;
            const uint32_t *rw = rank32 + w * Lh;
            uint32_t g = __vmaxu2(d[0], rw[roff[0]]);
#pragma unroll
            for (int i = 1; i + 1 < NV; i += 2)
                g = __vimin3_u16x2(g, __vmaxu2(d[i], rw[roff[i]]), __vmaxu2(d[i + 1], rw[roff[i + 1]]));
            if (!(NV & 1)) g = __vminu2(g, __vmaxu2(d[NV - 1], rw[roff[NV - 1]]));
            const uint32_t S2 = P | (1u << w);
            const uint32_t row = a.rowoff[S2] + (uint32_t)__popc(S2 & ((1u << w) - 1u)) - a.row0;
            g32[row * Lh + cw] = g;
        }
    }
}

__global__ void __launch_bounds__(kBatchThreads, kBatchBlocksPerSm)
k_batch(int64_t B, int L, int k, const uint64_t *__restrict__ g_bits,
        const uint64_t *__restrict__ g_mem, const uint64_t *__restrict__ g_cap,
        const uint32_t *__restrict__ g_bw, double *__restrict__ o_beta, int32_t *__restrict__ o_m,
        int32_t *__restrict__ o_cuts, int32_t *__restrict__ o_place, int8_t *__restrict__ o_status)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const BatchLayout lay = batch_layout(L, k);
    uint64_t *M = reinterpret_cast<uint64_t *>(smem + lay.M);
    uint64_t *cap = reinterpret_cast<uint64_t *>(smem + lay.cap);
    uint64_t *s_bits = reinterpret_cast<uint64_t *>(smem + lay.bits);
    uint64_t *s_sorted = reinterpret_cast<uint64_t *>(smem + lay.sbits);
    uint32_t *s_bw = reinterpret_cast<uint32_t *>(smem + lay.bw);
    uint32_t *ubw = reinterpret_cast<uint32_t *>(smem + lay.ubw);
    int16_t *uord = reinterpret_cast<int16_t *>(smem + lay.uord);  // lists by ascending bandwidth
    uint32_t *rowoff = reinterpret_cast<uint32_t *>(smem + lay.rowoff);
    uint32_t *loff = reinterpret_cast<uint32_t *>(smem + lay.loff);    // first compact row of each level
    uint32_t *rowinfo = reinterpret_cast<uint32_t *>(smem + lay.rowinfo);
    uint16_t *mlist = reinterpret_cast<uint16_t *>(smem + lay.mlist);  // masks by (popcount, value)
    uint32_t *moff = reinterpret_cast<uint32_t *>(smem + lay.moff);    // first entry of each popcount
    uint16_t *dp = reinterpret_cast<uint16_t *>(smem + lay.dp);        // [compact row][L]
    uint16_t *gbuf = reinterpret_cast<uint16_t *>(smem + lay.g);       // [row within level][L]
    uint16_t *rank = reinterpret_cast<uint16_t *>(smem + lay.rank);    // [v][w][c]
    uint16_t *rk = reinterpret_cast<uint16_t *>(smem + lay.rk);        // [U][L]
    uint32_t *cnt = reinterpret_cast<uint32_t *>(smem + lay.cnt);      // [U][L]
    unsigned long long *skey = reinterpret_cast<unsigned long long *>(smem + lay.skey);  // quotient matrix
    int16_t *pair_u = reinterpret_cast<int16_t *>(smem + lay.pair_u);
    int16_t *pos = reinterpret_cast<int16_t *>(smem + lay.pos);
    int16_t *lo = reinterpret_cast<int16_t *>(smem + lay.lo);
    __shared__ unsigned long long s_key[kBatchWarps];
    __shared__ unsigned long long s_best;
    __shared__ int s_bad, s_U;

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t nm = 1u << k;
    const int Ls = (L + 1) & ~1, Lh = Ls >> 1;  // row stride (even) and words per row
    // a thread's items advance by the block size: (row, column) moves by (dr, dc) with one carry
    const int drA = kBatchThreads / Lh, dcA = kBatchThreads - drA * Lh;
    const double kInf = __longlong_as_double(0x7FF0000000000000ll);

    // ---- instance-independent tables -------------------------------------------------------
    // Compact rows are ordered by (popcount, mask, node), so the rows of a level are contiguous.
    // rowoff[S] = compact row of (S, lowest node of S); loff[j] = first row of level j.
    if (tid <= k + 1) {
        uint32_t cnt = 0;  // rows of all masks with popcount below tid
        uint32_t masks = 0;
        for (uint32_t S = 0; S < nm; ++S) {
            cnt += (__popc(S) < tid) ? __popc(S) : 0;
            masks += (__popc(S) < tid);
        }
        loff[tid] = cnt;
        moff[tid] = masks;
    }
    __syncthreads();
    for (uint32_t S = tid; S < nm; S += kBatchThreads) {
        const int pc = __popc(S);
        uint32_t before = 0;  // masks of the same popcount below S
        for (uint32_t T = 0; T < S; ++T) before += (__popc(T) == pc);
        rowoff[S] = loff[pc] + before * pc;
        mlist[moff[pc] + before] = (uint16_t)S;
    }
    __syncthreads();
    for (uint32_t S = 1 + tid; S < nm; S += kBatchThreads) {
        int wi = 0;
        for (uint32_t rem = S; rem; rem &= rem - 1, ++wi) {
            const int w = __ffs(rem) - 1;
            const uint32_t P = S & ~(1u << w);
            rowinfo[rowoff[S] + wi] = info_pack(P, w, P ? rowoff[P] : 0u);
        }
    }
    const int jmax = k < L ? k : L;

    for (int64_t inst = blockIdx.x; inst < B; inst += gridDim.x) {
        const uint64_t *bits = g_bits + inst * L;
        const uint64_t *mem = g_mem + inst * L;
        const uint32_t *bw = g_bw + inst * k * k;
        __syncthreads();
        // ---- 1. stage inputs, prefix sums, windows ----
        for (int i = tid; i < L; i += kBatchThreads) {
            s_bits[i] = bits[i];
            M[i + 1] = mem[i];
        }
        for (int i = tid; i < k * k; i += kBatchThreads) s_bw[i] = bw[i];
        if (tid < k) cap[tid] = g_cap[inst * k + tid];
        if (tid == 0) s_bad = 0;
        __syncthreads();
        if (tid == 0) {
            uint64_t acc = 0;
            M[0] = 0;
            for (int i = 1; i <= L; ++i) {
                if (M[i] > ~0ull - acc) s_bad = 1;  // the 64-bit sum would wrap: PP_ERR_LIMIT, as in pp_problem_create
                acc += M[i];
                M[i] = acc;
            }
        }
        // distinct usable bandwidths in order of first appearance, one thread per node pair:
        // first_p[p] = earliest pair with the same bandwidth, then its index among the firsts
        for (int p = tid; p < k * k; p += kBatchThreads) {
            const int v = p / k, w = p - v * k;
            const uint32_t b = s_bw[p];
            int first = -1;
            if (v != w && b != 0) {
                first = p;
                for (int p2 = p - 1; p2 >= 0; --p2) {
                    const int v2 = p2 / k;
                    if (v2 != p2 - v2 * k && s_bw[p2] == b) first = p2;
                }
            }
            pair_u[p] = (int16_t)first;  // provisional: pair index of the first occurrence
        }
        // layers in ascending order of bits (ties by index)
        for (int c = tid; c < L; c += kBatchThreads) {
            const uint64_t b = s_bits[c];
            int p = 0;
            for (int o = 0; o < L; ++o) {
                const uint64_t x = s_bits[o];
                p += (x < b) || (x == b && o < c);
            }
            pos[c] = (int16_t)p;
            s_sorted[p] = b;
            if (b >= PP_MAX_BITS) s_bad = 1;
        }
        for (int i = tid; i < k * k; i += kBatchThreads)
            if (s_bw[i] >= PP_MAX_KBPS) s_bad = 1;
        __syncthreads();
        for (int p = tid; p < k * k; p += kBatchThreads) {
            const int first = pair_u[p];
            int u = -1;
            if (first >= 0) {
                u = 0;
                for (int p2 = 0; p2 < first; ++p2) u += (pair_u[p2] == p2);
                if (first == p) ubw[u] = s_bw[p];
            }
            reinterpret_cast<int16_t *>(cnt)[p] = (int16_t)u;  // staged: pair_u is still being read
        }
        if (tid == kBatchThreads - 1) {
            int U = 0;
            for (int p2 = 0; p2 < k * k; ++p2) U += (pair_u[p2] == p2);
            s_U = U;
        }
        __syncthreads();
        for (int p = tid; p < k * k; p += kBatchThreads) pair_u[p] = reinterpret_cast<int16_t *>(cnt)[p];
        const int U = s_U;
        for (int u = tid; u < U; u += kBatchThreads) {  // distinct values: positions are unique
            int at = 0;
            for (int u2 = 0; u2 < U; ++u2) at += (ubw[u2] < ubw[u]);
            uord[at] = (int16_t)u;
        }
        for (int e = tid; e < k * Ls; e += kBatchThreads) {
            const int w = e / Ls, c2 = e - w * Ls;
            int c = c2;  // step down while the segment starting at layer c (previous cut c-1) fits
            while (c2 < L && c > 0 && M[c2 + 1] - M[c] <= cap[w]) --c;
            lo[e] = (int16_t)c;  // the pad of an odd L keeps c2: an empty window
        }
        // ---- 2. quotients and their ranks ----
        // Rank = 1 + number of quotients strictly below.  The quotients form a matrix whose rows (one
        // per distinct bandwidth, widest link first) and columns (layers by ascending bits) both
        // ascend, so the count for one entry is a staircase walk: in every row step left while the
        // element is not below the entry, add the column reached, go down a row.  A walk takes
        // exactly U + L steps (row U is a row of +inf that empties the column counter), each one
        // shared-memory load and a few selects, and needs no barrier.  Positive doubles order like
        // their bit patterns.
        {
            const int n = U * L;
            unsigned long long *K = skey;  // K[1 + r * L + i]; K[0] is only read behind the j > 0 test
            __syncthreads();               // uord is complete
            for (int e = tid; e < (U + 1) * L; e += kBatchThreads) {
                const int r = e / L, i = e - r * L;
                K[1 + e] = r < U ? (unsigned long long)__double_as_longlong(__ddiv_rn(
                                       (double)s_sorted[i], (double)ubw[uord[U - 1 - r]]))
                                 : ~0ull;
            }
            if (tid == 0) K[0] = 0ull;
            __syncthreads();
            const int steps = U + L;
            for (int e = tid; e < n; e += kBatchThreads) {
                const int r0 = e / L, i = e - r0 * L;
                const unsigned long long x = K[1 + e];
                int j = L, p = L, acc = 0;  // p = r * L + j: the element left of column j in row r
#pragma unroll 4
                for (int st = 0; st < steps; ++st) {
                    const bool ge = j > 0 && K[p] >= x;
                    acc += ge ? 0 : j;
                    p += ge ? -1 : L;
                    j -= ge ? 1 : 0;
                }
                rk[uord[U - 1 - r0] * L + i] = (uint16_t)(1 + acc);
            }
        }
        __syncthreads();
        for (int e = tid; e < k * k * Ls; e += kBatchThreads) {
            const int r = e / Ls, c = e - r * Ls;
            const int u = pair_u[r];
            rank[e] = (u < 0 || c >= L) ? kInf16 : rk[u * L + pos[c]];
        }
        __syncthreads();  // the per-entry ranks share their bytes with the state table
        // base frontier
        for (int e = tid; e < k * Ls; e += kBatchThreads) {
            const int v = e / Ls, c = e - v * Ls;
            dp[(size_t)rowoff[1u << v] * Ls + c] = (c < L && M[c + 1] <= cap[v]) ? (uint16_t)0 : kInf16;
        }
        __syncthreads();
        // ---- 3. levels ----
        for (int j = 2; j <= k; ++j) {
            const uint32_t row0 = loff[j], nrows = loff[j + 1] - row0;
            if (j > jmax) {
                for (uint32_t it = tid; it < nrows * Ls; it += kBatchThreads) dp[(size_t)row0 * Ls + it] = kInf16;
                __syncthreads();
                continue;
            }
            // phase A: thread <-> (source mask P, word of two positions); the words of P's rows stay
            // in registers for all target nodes
            {
                const BatchRelaxArgs ra = {dp, gbuf, rank, rowoff, mlist + moff[j - 1], moff[j] - moff[j - 1],
                                           row0, k, Lh};
                switch (j - 1) {
#define PP_CASE(N) case N: batch_relax<N>(ra, tid); break;
                    PP_CASE(1) PP_CASE(2) PP_CASE(3) PP_CASE(4) PP_CASE(5) PP_CASE(6)
                    PP_CASE(7) PP_CASE(8) PP_CASE(9) PP_CASE(10) PP_CASE(11)
#undef PP_CASE
                    default: break;
                }
            }
            __syncthreads();
            {  // phase B: thread <-> (row, word): the windows of two neighbouring positions
               // [l0, c2-1] and [l1, c2] share the run [l1, c2-1], scanned once
                int rr = tid / Lh, cw = tid - rr * Lh;
                while (rr < (int)nrows) {
                    const int w = (rowinfo[row0 + rr] >> 12) & 15;
                    const uint16_t *gr = gbuf + rr * Ls;
                    const int c2 = 2 * cw;
                    const uint32_t ll = reinterpret_cast<const uint32_t *>(lo)[w * Lh + cw];  // starts of c2, c2+1
                    const int l0 = (int)(ll & 0xFFFFu), l1 = (int)(ll >> 16);
                    uint32_t head = kInf16, common = kInf16;
                    // one plain loop over [l0, c2-1]: the runs are a few positions long and differ from
                    // lane to lane, so unrolled and split loops only add instructions
#pragma unroll 1
                    for (int c = l0; c < c2; ++c) {
                        const uint32_t x = gr[c];
                        if (c < l1) head = min(head, x); else common = min(common, x);
                    }
                    const uint32_t out0 = min(head, common);
                    const uint32_t out1 = l1 <= c2 ? min(common, (uint32_t)gr[c2]) : (uint32_t)kInf16;
                    reinterpret_cast<uint32_t *>(dp)[(row0 + rr) * Lh + cw] = out0 | (out1 << 16);
                    rr += drA;
                    cw += dcA;
                    if (cw >= Lh) { cw -= Lh; ++rr; }
                }
            }
            __syncthreads();
        }
        // ---- 4. final state: smallest (value, popcount, mask, node) at c = L-1 ----
        unsigned long long key = kNoBest;
        for (uint32_t row = tid; row < loff[k + 1]; row += kBatchThreads) {
            const uint32_t x = dp[(size_t)row * Ls + (L - 1)];
            if (x == kInf16) continue;
            const uint32_t info = rowinfo[row];
            const int w = (info >> 12) & 15;
            const uint32_t S = (info & 0xFFFu) | (1u << w);
            const unsigned long long cand = pack_best(x, __popc(S), S, w);
            key = cand < key ? cand : key;
        }
        for (int o = 16; o; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, key, o);
            key = other < key ? other : key;
        }
        if (lane == 0) s_key[wid] = key;
        __syncthreads();
        if (tid == 0) {
            for (int i = 1; i < kBatchWarps; ++i) key = s_key[i] < key ? s_key[i] : key;
            s_best = key;
        }
        __syncthreads();
        key = s_best;
        const int bad = s_bad;
        int32_t *cuts = o_cuts ? o_cuts + inst * (k - 1) : nullptr;
        int32_t *place = o_place + inst * k;
        if (tid < k) place[tid] = -1;
        if (cuts && tid < k - 1) cuts[tid] = -1;
        __syncthreads();
        if (bad || key == kNoBest) {
            if (tid == 0) {
                o_beta[inst] = kInf;
                o_m[inst] = 0;
                o_status[inst] = bad ? (int8_t)PP_ERR_LIMIT : (int8_t)PP_INFEASIBLE;
            }
            continue;
        }
        if (wid == 0) {  // value of the winning rank, then the backtrack, by one warp
            const uint32_t rstar = (uint32_t)(key >> 30);
            const int m = (int)((key >> 25) & 31);
            uint32_t S = (uint32_t)((key >> 5) & 0xFFFFF);
            int w = (int)(key & 31), c2 = L - 1;
            double bstar = 0.0;
            if (rstar != 0) {
                // an entry of the rank table that carries the winning rank names a (node pair, layer)
                // whose quotient is beta* (equal ranks hold equal doubles)
                int found = -1;
                for (int e = lane; e < k * k * Ls; e += 32)
                    if (rank[e] == rstar) found = e;
                for (int o = 16; o; o >>= 1) {
                    const int other = __shfl_xor_sync(0xFFFFFFFFu, found, o);
                    found = other > found ? other : found;
                }
                const int r = found / Ls, c = found - r * Ls;
                bstar = __ddiv_rn((double)s_sorted[pos[c]], (double)ubw[pair_u[r]]);
            }
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
                const uint32_t P = S & ~(1u << w);
                const int l0 = lo[w * Ls + c2];
                unsigned int pick = 0xFFFFFFFFu;
                for (int it = lane; it < (c2 - l0) * k; it += 32) {
                    const int c = l0 + it / k, v = it - (it / k) * k;
                    if (!((P >> v) & 1u)) continue;
                    const uint32_t a = dp[(size_t)(rowoff[P] + __popc(P & ((1u << v) - 1u))) * Ls + c];
                    const uint32_t b = rank[(v * k + w) * Ls + c];
                    const uint32_t mx = a > b ? a : b;
                    if (mx <= rstar) {
                        const unsigned int kk = ((unsigned)c << 5) | (unsigned)v;
                        pick = kk < pick ? kk : pick;
                    }
                }
                for (int o = 16; o; o >>= 1) {
                    const unsigned int other = __shfl_xor_sync(0xFFFFFFFFu, pick, o);
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
