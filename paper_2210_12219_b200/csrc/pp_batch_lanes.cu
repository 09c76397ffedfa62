// Many-instance exact search, one instance per lane.
//
// The block-per-instance kernel (pp_batch.cu) spends most of its instructions on addressing: a
// thread owns one word of one row and has to find out which.  Here a warp owns one source mask P of
// 32 instances at once, lane <-> instance.  Every lane then walks the same masks, nodes and cut
// positions, so all of that is uniform and unrolled, and the only per-lane data are the states, the
// gamma ranks and the window lengths.  Those live in global memory (L2-resident for a chunk of a
// few thousand instances), instance-minor: the 32 lanes of a warp read 32 neighbouring words.
//
// Per chunk of instances:
//   1. k_lanes_prep, one warp per instance: staging, windows, the ranking of gamma (Eq. 3); writes
//      the instance's column of the rank table, the window lengths, the base frontier and the best
//      single-node plan;
//   2. one launch per popcount level, k_lanes_level<NV, LH>: a warp takes (group of 32 instances,
//      source mask P of NV nodes), keeps the NV rows of P in registers (two cut positions per 32-bit
//      word, LH words per row), and for every node w outside P forms
//      g[c] = min_v max(dp[P][v][c], rank[v][w][c]) with packed 16-bit min/max, takes the window
//      minimum over [lo_w(c'), c'-1] from a sparse table of g in the lane's own column of shared
//      memory (the one place where a lane needs an index of its own), stores the row of (P + w, w), and keeps the smallest final state
//      (value, popcount, mask, node), merged into the instance's key with one atomic per lane;
//   3. k_lanes_back, one warp per instance: the value of the winning rank and the backtrack by the
//      threshold rule, lanes over the candidates.
// Same recurrence, final choice and backtrack rule as the single-instance path (pp_sweep.cu).
#include "pp_internal.cuh"

namespace pp {

namespace {

constexpr int kLevelWarps = 4;
constexpr int kLevelFourBlocks = 5;  // source masks of up to this many nodes: registers capped for four blocks per SM
constexpr int kPrepWarps = 4;
constexpr int kFlagLimit = 1;     // BatchLanes::flag: an input beyond the limits
constexpr int kFlagDeferred = 2;  // ... the first preparing pass left the ranking to the second
constexpr int kWalks = 2;  // staircase walks a lane runs interleaved: the walk is a chain of dependent loads
constexpr int kBackWarps = 8;
constexpr int kLanesMinB = 64;  // below this the block-per-instance kernel keeps more of the GPU busy
constexpr int kLanesMaxK = 8;   // NV <= 7 rows of a source mask in registers
constexpr int kLanesMaxL = 32;  // LH <= 16 words per row

// Sparse table of one row g in a warp's shared memory: level s holds T_s[c] = min g[c - 2^s + 1 .. c],
// two positions per 32-bit word like the rows, word (s, wd) of lane l at byte ((s LH + wd) 32 + l) 4:
// every lane reads and writes its own bank.  Word kWinLevels * LH holds +inf.  A cell is named by
// its byte offset without the lane's part, which fits 16 bits.
constexpr int kWinLevels = 5;  // windows of up to 31 positions
__host__ __device__ inline uint32_t win_cell(int s, int pos, int LH)
{
    return (uint32_t)((s * LH + (pos >> 1)) * 128 + (pos & 1) * 2);
}
__host__ __device__ inline size_t win_bytes_per_warp(int LH) { return (size_t)(kWinLevels * LH + 1) * 128; }

// Checked access to one of the tables of BatchLanes: in the bounds-checking build an address outside
// [base, base + words) is recorded in the error word and the access skipped (a load gives +inf); in
// the normal build PP_IN_BOUNDS is `true` and these are plain loads and stores.
__device__ __forceinline__ uint32_t ld_table(const BatchLanes &t, const uint32_t *p, const uint32_t *base, size_t words)
{
    return PP_IN_BOUNDS(t, (size_t)(p - base), words) ? *p : 0xFFFFFFFFu;
}
__device__ __forceinline__ void st_table(const BatchLanes &t, uint32_t *p, const uint32_t *base, size_t words, uint32_t v)
{
    if (PP_IN_BOUNDS(t, (size_t)(p - base), words)) *p = v;
}

// Shared memory of one warp of the preparing kernel (byte offsets; every part 16-byte aligned).
struct PrepLayout {
    size_t K, M, bits, sorted, cap, bw, ubw, rk, pair_u, rowu, pos, total;
    int Ks;  // row stride of the quotient matrix in keys: a sentinel in front of the L quotients
};

__host__ __device__ inline PrepLayout prep_layout(int L, int ucap)
{
    PrepLayout p;
    const size_t U = (size_t)ucap;  // distinct bandwidths the quotient matrix has room for
    size_t o = 0;
    auto take = [&o](size_t bytes) { size_t at = o; o = (o + bytes + 15) & ~(size_t)15; return at; };
    p.Ks = L + 1;
    p.K = take((U + 1) * (size_t)p.Ks * 8);
    p.M = take(33 * 8);
    p.bits = take(32 * 8);
    p.sorted = take(32 * 8);
    p.cap = take(8 * 8);
    p.bw = take(64 * 4);
    p.ubw = take(64 * 4);
    p.rk = take((U * L + 1) * 2);
    p.pair_u = take(64);
    p.rowu = take(64);
    p.pos = take(32);
    p.total = o;
    return p;
}

// One warp per instance, lane <-> layer (L <= 32) or node pair (k * k <= 64, two per lane): staging,
// the windows, the ranking of gamma (Eq. 3), and the instance's column of the tables of BatchLanes.
//   * layers ordered by bits (ties by index), distinct usable bandwidths listed in order of first
//     appearance, as in the block-per-instance kernel;
//   * window start lo_w(c2) by a branch-free binary search over the memory prefix sums;
//   * rank = 1 + number of quotients strictly below.  The quotients form a matrix whose rows (one
//     per distinct bandwidth, widest link first) and columns (layers by ascending bits) both ascend,
//     so the count for one entry is a staircase walk: in every row step left while the element is
//     not below the entry, add the column reached, go down a row.  Keys are the bit patterns of the
//     quotients (positive doubles order like them) plus one, so that a zero in front of every row
//     stops the walk to the left without a test; row U holds the largest key and empties the column
//     counter; a walk takes exactly U + L steps.  A lane runs several walks interleaved.
// The matrix is the bulk of a warp's shared memory, and the walks are chains of dependent loads that
// want many warps in flight, so the kernel runs twice: the first pass has room for k (k - 1) / 2
// distinct bandwidths (every symmetric network) and marks an instance that has more; the second pass,
// with room for k (k - 1), takes only the marked ones and returns at once from all others.
__global__ void __launch_bounds__(kPrepWarps * 32)
k_lanes_prep(const BatchLanes t, const int64_t B, const int L, const int k, const uint64_t *__restrict__ g_bits,
             const uint64_t *__restrict__ g_mem, const uint64_t *__restrict__ g_cap,
             const uint32_t *__restrict__ g_bw, const int ucap, const int second_pass)
{
    extern __shared__ __align__(16) unsigned char smem_prep[];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const PrepLayout lay = prep_layout(L, ucap);
    unsigned char *base = smem_prep + (size_t)wid * lay.total;
    unsigned long long *K = reinterpret_cast<unsigned long long *>(base + lay.K);
    unsigned long long *M = reinterpret_cast<unsigned long long *>(base + lay.M);
    unsigned long long *s_bits = reinterpret_cast<unsigned long long *>(base + lay.bits);
    unsigned long long *s_sorted = reinterpret_cast<unsigned long long *>(base + lay.sorted);
    unsigned long long *s_cap = reinterpret_cast<unsigned long long *>(base + lay.cap);
    uint32_t *s_bw = reinterpret_cast<uint32_t *>(base + lay.bw);
    uint32_t *ubw = reinterpret_cast<uint32_t *>(base + lay.ubw);
    uint16_t *rk = reinterpret_cast<uint16_t *>(base + lay.rk);
    int8_t *pair_u = reinterpret_cast<int8_t *>(base + lay.pair_u);
    uint8_t *rowu = base + lay.rowu;
    uint8_t *pos = base + lay.pos;
    const int Ks = lay.Ks, LH = t.LH, kk = k * k;
    const uint32_t FULL = 0xFFFFFFFFu;
    // floor(x / k) for x < 64 and floor(x / L) for x < k (k-1) L <= 1792 by a multiplication
    const uint32_t recip_k = (65536u + (uint32_t)k - 1u) / (uint32_t)k;
    const uint32_t recip_L = (65536u + (uint32_t)L - 1u) / (uint32_t)L;
    for (int64_t inst = (int64_t)blockIdx.x * kPrepWarps + wid; inst < B; inst += (int64_t)gridDim.x * kPrepWarps) {
        if (second_pass && !(t.flag[inst] & kFlagDeferred)) continue;  // ranked by the first pass
        __syncwarp();
        // ---- staging, prefix sums of the memory ----
        const unsigned long long b = lane < L ? g_bits[inst * L + lane] : 0ull;
        const unsigned long long mm = lane < L ? g_mem[inst * L + lane] : 0ull;
        const uint32_t bw0 = lane < kk ? g_bw[inst * kk + lane] : 0u;
        const uint32_t bw1 = lane + 32 < kk ? g_bw[inst * kk + lane + 32] : 0u;
        bool bad = b >= PP_MAX_BITS || bw0 >= PP_MAX_KBPS || bw1 >= PP_MAX_KBPS;
        unsigned long long x = mm;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long y = __shfl_up_sync(FULL, x, o);
            if (lane >= o) {
                if (y > ~0ull - x) bad = true;  // the 64-bit sum would wrap: PP_ERR_LIMIT
                x += y;
            }
        }
        if (lane == 0) M[0] = 0ull;
        M[lane + 1] = x;  // beyond L: the total, never read
        s_bits[lane] = b;
        s_bw[lane] = bw0;
        s_bw[lane + 32] = bw1;
        if (lane < k) s_cap[lane] = g_cap[inst * k + lane];
        bad = __any_sync(FULL, bad);
        __syncwarp();
        // ---- layers in ascending order of bits (ties by index) ----
        {
            int p = 0;
            for (int o = 0; o < L; ++o) {
                const unsigned long long xo = s_bits[o];
                p += (xo < b) || (xo == b && o < lane);
            }
            if (lane < L) {
                s_sorted[p] = b;
                pos[lane] = (uint8_t)p;
            }
        }
        // ---- distinct usable bandwidths in order of first appearance ----
        int U;
        {
            const int p0 = lane, p1 = lane + 32;
            const int v0 = (int)(((uint32_t)p0 * recip_k) >> 16), v1 = (int)(((uint32_t)p1 * recip_k) >> 16);
            const bool us0 = p0 < kk && v0 != p0 - v0 * k && bw0 != 0u;
            const bool us1 = p1 < kk && v1 != p1 - v1 * k && bw1 != 0u;
            int f0 = us0 ? p0 : -1, f1 = us1 ? p1 : -1;
            int v2 = 0, w2 = 0;
            for (int p2 = 0; p2 < kk; ++p2) {  // ascending: the first match stays
                const uint32_t b2 = s_bw[p2];
                const bool us2 = v2 != w2 && b2 != 0u;
                if (us2 && us0 && b2 == bw0 && p2 < f0) f0 = p2;
                if (us2 && us1 && b2 == bw1 && p2 < f1) f1 = p2;
                if (++w2 == k) { w2 = 0; ++v2; }
            }
            const bool first0 = us0 && f0 == p0, first1 = us1 && f1 == p1;
            const uint32_t m0 = __ballot_sync(FULL, first0), m1 = __ballot_sync(FULL, first1);
            const int n0 = __popc(m0);
            U = n0 + __popc(m1);
            auto index_of = [&](int f) {
                return f < 32 ? __popc(m0 & ((1u << f) - 1u)) : n0 + __popc(m1 & ((1u << (f - 32)) - 1u));
            };
            const int u0 = f0 >= 0 ? index_of(f0) : -1, u1 = f1 >= 0 ? index_of(f1) : -1;
            pair_u[p0] = (int8_t)u0;
            pair_u[p1] = (int8_t)u1;
            if (first0) ubw[u0] = bw0;
            if (first1) ubw[u1] = bw1;
        }
        __syncwarp();
        // rows of the quotient matrix: widest link first (the values of a column then ascend)
        for (int u = lane; u < U; u += 32) {
            const uint32_t mine = ubw[u];
            int r = 0;
            for (int u2 = 0; u2 < U; ++u2) r += ubw[u2] > mine;
            rowu[r] = (uint8_t)u;
        }
        // ---- windows, base frontier ----
        {
            uint32_t *lT = t.len + (size_t)(inst >> 5) * (size_t)(k * LH) * 32 + (inst & 31);
            uint32_t *tT = t.table + (size_t)(inst >> 5) * (size_t)t.rows * LH * 32 + (inst & 31);
            uint32_t *wT = t.win + (size_t)(inst >> 5) * (size_t)(k * 2 * LH) * 32 + (inst & 31);
            const unsigned long long Mc = M[lane + 1];  // memory of layers 0..lane
            for (int w = 0; w < k; ++w) {
                const unsigned long long capw = s_cap[w];
                // c* = number of prefix sums M[0..lane+1] below M[lane+1] - cap: the first start layer
                // from which the segment ending at this layer fits; window start = max(c* - 1, 0)
                const unsigned long long thr = Mc > capw ? Mc - capw : 0ull;
                int cs = 0;
#pragma unroll
                for (int step = 32; step; step >>= 1)
                    if (cs + step <= lane + 2 && M[cs + step - 1] < thr) cs += step;
                const int lo = cs > 0 ? cs - 1 : 0;
                const uint32_t len = lane < L ? (uint32_t)(lane - lo) : 0u;
                const uint32_t inf = (lane < L && Mc <= capw) ? 0u : 0xFFFFu;
                const uint32_t len0 = __shfl_sync(FULL, len, 2 * lane), len1 = __shfl_sync(FULL, len, 2 * lane + 1);
                const uint32_t inf0 = __shfl_sync(FULL, inf, 2 * lane), inf1 = __shfl_sync(FULL, inf, 2 * lane + 1);
                {
                    // window [lo, lane - 1] of length len >= 1 = union of the two runs of 2^s positions
                    // that end at lane - 1 and that start at lo, s = floor(log2 len): their sparse-table
                    // cells; an empty window reads the cell that holds +inf
                    uint32_t code = win_cell(kWinLevels, 0, LH) * 0x00010001u;
                    if (len != 0u) {
                        const int sl = 31 - __clz((int)len);
                        code = win_cell(sl, lane - 1, LH) | (win_cell(sl, lo + (1 << sl) - 1, LH) << 16);
                    }
                    // position 0 has no window: its entry carries the highest level this node's windows read
                    const uint32_t longest = __reduce_max_sync(FULL, len);
                    if (lane == 0) code = longest > 1u ? (uint32_t)(31 - __clz((int)longest)) : 0u;
                    if (lane < 2 * LH) st_table(t, wT + (size_t)(w * 2 * LH + lane) * 32, t.win, t.win_words, code);
                }
                if (lane < LH) {
                    st_table(t, lT + (size_t)(w * LH + lane) * 32, t.len, t.len_words, lane < 16 ? len0 | (len1 << 16) : 0u);
                    st_table(t, tT + ((size_t)t.rowoff[1u << w] * LH + lane) * 32, t.table, t.table_words,
                             lane < 16 ? inf0 | (inf1 << 16) : 0xFFFFFFFFu);
                }
            }
            if (lane == 0) {
                unsigned long long best = kNoBest;
                for (int v = k - 1; v >= 0; --v)
                    if (M[L] <= s_cap[v]) best = pack_best(0u, 1, 1u << v, v);
                t.key[inst] = best;
                t.flag[inst] = (int8_t)((bad ? kFlagLimit : 0) | (U > ucap ? kFlagDeferred : 0));
            }
        }
        if (U > ucap) continue;  // more distinct bandwidths than this pass has room for: left to the second pass
        __syncwarp();
        // ---- quotient matrix ----
        for (int r = 0; r <= U; ++r) {
            unsigned long long key = ~0ull;
            if (r < U)
                key = 1ull + (unsigned long long)__double_as_longlong(
                                 __ddiv_rn((double)s_sorted[lane < L ? lane : 0], (double)ubw[rowu[r]]));
            if (lane < L) K[r * Ks + 1 + lane] = key;
            if (lane == 0) K[r * Ks] = 0ull;
        }
        __syncwarp();
        // ---- ranks ----
        {
            // The column counter is not kept: a step down from row r at column j leaves from byte
            // offset 8 (r Ks + j), so the sum of the offsets of the U steps down is
            // 8 (Ks U (U - 1) / 2 + sum of the columns).
            const int n = U * L, steps = U + L;
            const unsigned char *Kb = reinterpret_cast<const unsigned char *>(K);
            const int down = Ks * 8, start = L * 8;  // the last quotient of row 0
            const int rows_part = Ks * (U * (U - 1) / 2);
            for (int e0 = 0; e0 < n; e0 += 32 * kWalks) {
                unsigned long long x[kWalks];
                int p[kWalks], sum[kWalks], cell[kWalks];
#pragma unroll
                for (int q = 0; q < kWalks; ++q) {
                    const int e = e0 + 32 * q + lane;
                    const int r = (int)(((uint32_t)e * recip_L) >> 16), i = e - r * L;
                    // an idle lane walks with the smallest key: left along row 0, then down the zeros
                    x[q] = e < n ? K[r * Ks + 1 + i] : 1ull;
                    cell[q] = e < n ? rowu[r] * L + i : -1;
                    p[q] = start;
                    sum[q] = 0;
                }
#pragma unroll 2
                for (int st = 0; st < steps; ++st) {
#pragma unroll
                    for (int q = 0; q < kWalks; ++q) {
                        const bool ge = *reinterpret_cast<const unsigned long long *>(Kb + p[q]) >= x[q];
                        sum[q] += ge ? 0 : p[q];
                        p[q] += ge ? -8 : down;
                    }
                }
#pragma unroll
                for (int q = 0; q < kWalks; ++q)
                    if (cell[q] >= 0) rk[cell[q]] = (uint16_t)(1 + (sum[q] >> 3) - rows_part);
            }
        }
        __syncwarp();
        // ---- rank table, two positions per word: rank[v][w][c] = rank of (bandwidth of v -> w, layer c) ----
        {
            uint32_t *rT = t.rank + (size_t)(inst >> 5) * (size_t)(kk * LH) * 32 + (inst & 31);
            const int c0 = 2 * lane, c1 = 2 * lane + 1;
            const int q0 = c0 < L ? pos[c0] : 0, q1 = c1 < L ? pos[c1] : 0;
            for (int pr = 0; pr < kk; ++pr) {
                const int u = pair_u[pr];
                uint32_t word = 0xFFFFFFFFu;
                if (u >= 0) {
                    const uint32_t a = c0 < L ? rk[u * L + q0] : 0xFFFFu;
                    const uint32_t c = c1 < L ? rk[u * L + q1] : 0xFFFFu;
                    word = a | (c << 16);
                }
                if (lane < LH) st_table(t, rT + (size_t)(pr * LH + lane) * 32, t.rank, t.rank_words, word);
            }
        }
    }
}

__device__ __forceinline__ void st_shared_u32(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_shared_u16(uint32_t addr)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr) : "memory");
    return v;
}

template <int NV, int LH>
__global__ void __launch_bounds__(kLevelWarps * 32, NV <= kLevelFourBlocks ? 4 : 3)
k_lanes_level(const BatchLanes t, const int64_t B, const int k, const int L, const int split)
{
    // Launched as a programmatic dependent of the kernel before it: nothing is read before that
    // kernel is complete, and the next one may be scheduled as soon as this one's blocks retire.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    const int lane = threadIdx.x & 31;
    extern __shared__ __align__(16) unsigned char smem_level[];
    const uint32_t sbase = (uint32_t)__cvta_generic_to_shared(smem_level) +
                           (uint32_t)((threadIdx.x >> 5) * win_bytes_per_warp(LH)) + (uint32_t)lane * 4u;
    // A state of j segments ends at layer j - 1 at the earliest: rows of this level's sources (NV
    // nodes) are +inf before position NV - 1 and the rows written here before position NV.  Words
    // that hold only such positions are neither read, computed nor written, here and in the next
    // level alike; their cells of the sparse table are set to +inf once.
    constexpr int W0 = (NV - 1) / 2;  // first word of a source row that can hold a state
    constexpr int C0 = NV;            // first position of a target row that can
    constexpr int O0 = NV / 2;        // its word: the first one stored (the next level's W0)
    st_shared_u32(sbase + win_cell(kWinLevels, 0, LH), 0xFFFFFFFFu);
#pragma unroll
    for (int sl = 0; sl < kWinLevels; ++sl)
#pragma unroll
        for (int wd = 0; wd < W0; ++wd) st_shared_u32(sbase + win_cell(sl, 2 * wd, LH), 0xFFFFFFFFu);
    const uint32_t nmasks = t.moff[NV + 1] - t.moff[NV];
    const int64_t G = (B + 31) >> 5;
    // a level with few source masks gives the targets of one mask to `split` warps
    const int64_t items = G * nmasks * split;
    const uint32_t full = (1u << k) - 1u;
    const int wfin = (L - 1) >> 1, sfin = ((L - 1) & 1) * 16;
    for (int64_t item = (int64_t)blockIdx.x * kLevelWarps + (threadIdx.x >> 5); item < items;
         item += (int64_t)gridDim.x * kLevelWarps) {
        const int64_t g = item / (nmasks * split);
        const uint32_t within = (uint32_t)(item - g * (nmasks * split));
        const uint32_t P = t.mlist[t.moff[NV] + within / (uint32_t)split];
        const int part = (int)(within % (uint32_t)split);
        // lanes past the end of the batch read the last instance's column and store to their own
        const int64_t left = B - g * 32;
        const int valid = left < 32 ? (int)left : 32;
        const int col = lane < valid ? lane : valid - 1;
        const uint32_t *tab = t.table + (size_t)g * t.rows * (LH * 32) + col;
        uint32_t *tabw = t.table + (size_t)g * t.rows * (LH * 32) + lane;
        const uint32_t *rk = t.rank + (size_t)g * (size_t)(k * k) * (LH * 32) + col;
        const uint32_t *wn = t.win + (size_t)g * (size_t)(k * 2) * (LH * 32) + col;
        uint32_t d[NV][LH];
        int vs[NV];
        {
            const uint32_t row0 = t.rowoff[P];
            uint32_t rem = P;
#pragma unroll
            for (int vi = 0; vi < NV; ++vi) {
                vs[vi] = __ffs(rem) - 1;
                rem &= rem - 1;
#pragma unroll
                for (int wd = W0; wd < LH; ++wd)
                    d[vi][wd] = ld_table(t, tab + ((size_t)(row0 + vi) * LH + wd) * 32, t.table, t.table_words);
            }
        }
        unsigned long long key = kNoBest;
        int turn = part;
        for (uint32_t wrem = full & ~P; wrem; wrem &= wrem - 1) {
            if (turn-- != 0) continue;  // another warp's target
            turn = split - 1;
            const int w = __ffs(wrem) - 1;
            // the window cells of this node, asked for before anything else; position 0 has no window
            // and its entry carries the highest level of the sparse table this (instance, node) reads
            uint32_t cw[2 * LH];
            const uint32_t lvl = ld_table(t, wn + (size_t)(w * 2 * LH) * 32, t.win, t.win_words);
#pragma unroll
            for (int c2 = C0; c2 < 2 * LH; ++c2)
                cw[c2] = ld_table(t, wn + (size_t)(w * 2 * LH + c2) * 32, t.win, t.win_words);
            uint32_t gg[LH];
            {
                const uint32_t *r0 = rk + (size_t)((vs[0] * k + w) * LH) * 32;
#pragma unroll
                for (int wd = W0; wd < LH; ++wd) gg[wd] = __vmaxu2(d[0][wd], ld_table(t, r0 + wd * 32, t.rank, t.rank_words));
            }
#pragma unroll
            for (int vi = 1; vi + 1 < NV; vi += 2) {
                const uint32_t *r1 = rk + (size_t)((vs[vi] * k + w) * LH) * 32;
                const uint32_t *r2 = rk + (size_t)((vs[vi + 1] * k + w) * LH) * 32;
#pragma unroll
                for (int wd = W0; wd < LH; ++wd)
                    gg[wd] = __vimin3_u16x2(gg[wd], __vmaxu2(d[vi][wd], ld_table(t, r1 + wd * 32, t.rank, t.rank_words)),
                                            __vmaxu2(d[vi + 1][wd], ld_table(t, r2 + wd * 32, t.rank, t.rank_words)));
            }
            if (!(NV & 1)) {
                const uint32_t *r1 = rk + (size_t)((vs[NV - 1] * k + w) * LH) * 32;
#pragma unroll
                for (int wd = W0; wd < LH; ++wd) gg[wd] = __vminu2(gg[wd], __vmaxu2(d[NV - 1][wd], ld_table(t, r1 + wd * 32, t.rank, t.rank_words)));
            }
            // Window minimum over [lo_w(c2), c2 - 1] for every c2: the sparse table of g goes to the
            // lane's column of shared memory, level s from level s - 1 by one packed minimum per word
            // (level 1 needs the row shifted by one position), up to the highest level a lane of this
            // warp reads; every cut position then reads the two cells the preparing kernel named for it.
            {
                const int top = (int)__reduce_max_sync(0xFFFFFFFFu, lvl);
                uint32_t cur[LH];
#pragma unroll
                for (int wd = W0; wd < LH; ++wd) {
                    st_shared_u32(sbase + win_cell(0, 2 * wd, LH), gg[wd]);
                    const uint32_t prev = wd > W0 ? gg[wd - 1] : 0xFFFFFFFFu;
                    cur[wd] = __vminu2(gg[wd], __byte_perm(prev, gg[wd], 0x5432));  // positions 2wd-1, 2wd
                    st_shared_u32(sbase + win_cell(1, 2 * wd, LH), cur[wd]);
                }
#pragma unroll
                for (int sl = 2; sl < kWinLevels; ++sl) {
                    if (sl > top) break;
                    const int shift = 1 << (sl - 2);  // words
#pragma unroll
                    for (int wd = LH - 1; wd >= W0; --wd) {  // downwards: cur[wd - shift] is still the level below
                        if (wd - shift >= W0) cur[wd] = __vminu2(cur[wd], cur[wd - shift]);
                        st_shared_u32(sbase + win_cell(sl, 2 * wd, LH), cur[wd]);
                    }
                }
            }
            uint32_t ob[2 * LH];
#pragma unroll
            for (int c2 = 2 * O0; c2 < 2 * LH; ++c2) {
                ob[c2] = 0xFFFFu;
                if (c2 >= C0) {
                    // (bounds-checking build: a cell outside the warp's table reads the +inf cell instead)
                    const uint32_t o1 = PP_IN_BOUNDS(t, cw[c2] & 0xFFFFu, win_bytes_per_warp(LH) - 126) ? cw[c2] & 0xFFFFu
                                                                                                       : win_cell(kWinLevels, 0, LH);
                    const uint32_t o2 = PP_IN_BOUNDS(t, cw[c2] >> 16, win_bytes_per_warp(LH) - 126) ? cw[c2] >> 16
                                                                                                 : win_cell(kWinLevels, 0, LH);
                    const uint32_t a = ld_shared_u16(sbase + o1), b2 = ld_shared_u16(sbase + o2);
                    ob[c2] = min(a, b2);
                }
            }
            const uint32_t S2 = P | (1u << w);
            const uint32_t row = t.rowoff[S2] + (uint32_t)__popc(S2 & ((1u << w) - 1u));
            uint32_t xw = 0xFFFFFFFFu;
#pragma unroll
            for (int wd = O0; wd < LH; ++wd) {
                const uint32_t o = ob[2 * wd] | (ob[2 * wd + 1] << 16);
                st_table(t, tabw + ((size_t)row * LH + wd) * 32, t.table, t.table_words, o);
                if (wd == wfin) xw = o;
            }
            const uint32_t x = (xw >> sfin) & 0xFFFFu;
            if (x != 0xFFFFu) {
                const unsigned long long cand = pack_best(x, NV + 1, S2, w);
                key = cand < key ? cand : key;
            }
        }
        if (key != kNoBest && lane < valid) atomicMin(&t.key[g * 32 + lane], key);
    }
}

// state or rank of one (row, position) of one instance's column
__device__ __forceinline__ uint32_t lanes_elem(const BatchLanes &t, const uint32_t *col, const uint32_t *base, size_t words,
                                               size_t row, int LH, int c)
{
    return (ld_table(t, col + (row * LH + (size_t)(c >> 1)) * 32, base, words) >> ((c & 1) * 16)) & 0xFFFFu;
}

__global__ void __launch_bounds__(kBackWarps * 32)
k_lanes_back(const BatchLanes t, const int64_t B, const int L, const int k, const uint64_t *__restrict__ g_bits,
             const uint32_t *__restrict__ g_bw, double *__restrict__ o_beta, int32_t *__restrict__ o_m,
             int32_t *__restrict__ o_cuts, int32_t *__restrict__ o_place, int8_t *__restrict__ o_status)
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const int LH = t.LH;
    const double kInf = __longlong_as_double(0x7FF0000000000000ll);
    __shared__ uint32_t s_len[kBackWarps][kLanesMaxK * 16];  // the instance's window lengths: one load fewer per step
    uint32_t *mylen = s_len[threadIdx.x >> 5];
    for (int64_t inst = (int64_t)blockIdx.x * kBackWarps + (threadIdx.x >> 5); inst < B;
         inst += (int64_t)gridDim.x * kBackWarps) {
        const size_t g = (size_t)(inst >> 5);
        const int col = (int)(inst & 31);
        const uint32_t *tab = t.table + g * t.rows * (size_t)(LH * 32) + col;
        const uint32_t *rk = t.rank + g * (size_t)(k * k) * (size_t)(LH * 32) + col;
        const uint32_t *ln = t.len + g * (size_t)k * (size_t)(LH * 32) + col;
        const unsigned long long key = t.key[inst];
        const int bad = t.flag[inst] & kFlagLimit;
        int32_t *cuts = o_cuts ? o_cuts + inst * (k - 1) : nullptr;
        int32_t *place = o_place + inst * k;
        if (lane < k) place[lane] = -1;
        if (cuts && lane < k - 1) cuts[lane] = -1;
        __syncwarp();
        for (int e = lane; e < k * LH; e += 32) mylen[e] = ld_table(t, ln + (size_t)e * 32, t.len, t.len_words);
        __syncwarp();
        if (bad || key == kNoBest) {
            if (lane == 0) {
                o_beta[inst] = kInf;
                o_m[inst] = 0;
                o_status[inst] = bad ? (int8_t)PP_ERR_LIMIT : (int8_t)PP_INFEASIBLE;
            }
            continue;
        }
        const uint32_t rstar = (uint32_t)(key >> 30);
        const int m = (int)((key >> 25) & 31);
        uint32_t S = (uint32_t)((key >> 5) & 0xFFFFF);
        int w = (int)(key & 31), c2 = L - 1;
        double bstar = 0.0;
        if (rstar != 0) {
            // an entry of the rank table that carries the winning rank names a (node pair, layer) whose
            // quotient is beta* (equal ranks hold equal doubles)
            int found = -1;
#pragma unroll 8
            for (int e = lane; e < k * k * LH; e += 32) {
                const uint32_t x = ld_table(t, rk + (size_t)e * 32, t.rank, t.rank_words);
                if ((x & 0xFFFFu) == rstar) found = 2 * e;
                if ((x >> 16) == rstar) found = 2 * e + 1;
            }
            for (int o = 16; o; o >>= 1) {
                const int other = __shfl_xor_sync(0xFFFFFFFFu, found, o);
                found = other > found ? other : found;
            }
            const int r = (found >> 1) / LH, c = 2 * ((found >> 1) - r * LH) + (found & 1);
            bstar = __ddiv_rn((double)g_bits[inst * L + c], (double)g_bw[inst * k * k + r]);
        }
        if (lane == 0) {
            o_beta[inst] = bstar;
            o_m[inst] = m;
            o_status[inst] = (int8_t)PP_OK;
#ifdef PP_DEBUG_BOUNDS
            if (*t.err != 0) o_status[inst] = (int8_t)PP_ERR_CUDA;  // an index left its table somewhere in this piece
#endif
        }
        for (int j = m - 1; j >= 0; --j) {
            if (lane == 0) {
                place[j] = w;
                if (j < m - 1) cuts[j] = c2;
            }
            if (j == 0) break;
            const uint32_t P = S & ~(1u << w);
            const int l0 = c2 - (int)((mylen[w * LH + (c2 >> 1)] >> ((c2 & 1) * 16)) & 0xFFFFu);
            const uint32_t prow = t.rowoff[P];
            const int np = __popc(P), total = (c2 - l0) * np;
            // candidates (position, node of P), lanes over all of them at once: the loads of a step are
            // independent, the smallest (position, node) that meets the threshold wins
            unsigned int pick = 0xFFFFFFFFu;
#pragma unroll 2
            for (int it = lane; it < total; it += 32) {
                const int ci = it / np, vi = it - ci * np;
                const int c = l0 + ci, v = (int)__fns(P, 0, vi + 1);
                // a state of np segments ends at layer np - 1 at the earliest; earlier positions were never written
                const uint32_t a = c >= np - 1 ? lanes_elem(t, tab, t.table, t.table_words, (size_t)prow + vi, LH, c) : 0xFFFFu;
                const uint32_t b = lanes_elem(t, rk, t.rank, t.rank_words, (size_t)(v * k + w), LH, c);
                const uint32_t mx = a > b ? a : b;
                const unsigned int kk = ((unsigned)c << 5) | (unsigned)v;
                if (mx <= rstar && kk < pick) pick = kk;
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

template <typename... Args, typename... Params>
cudaError_t launch_dependent(void (*kernel)(Params...), unsigned grid, unsigned block, size_t smem, cudaStream_t s,
                             Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <int LH>
cudaError_t launch_level(int nv, const BatchLanes &t, int64_t B, int k, int L, int split, unsigned grid, cudaStream_t s)
{
    switch (nv) {
#define PP_CASE(N) \
    case N: {                                                                                                  \
        const size_t sm = win_bytes_per_warp(LH) * kLevelWarps;                                                \
        cudaError_t e = cudaFuncSetAttribute(k_lanes_level<N, LH>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                             (int)sm);                                                          \
        if (e != cudaSuccess) return e;                                                                        \
        return launch_dependent(k_lanes_level<N, LH>, grid, kLevelWarps * 32, sm, s, t, B, k, L, split);       \
    }
        PP_CASE(1) PP_CASE(2) PP_CASE(3) PP_CASE(4) PP_CASE(5) PP_CASE(6) PP_CASE(7)
#undef PP_CASE
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool batch_lanes_takes(int64_t B, int L, int k)
{
    return B >= kLanesMinB && k >= 2 && k <= kLanesMaxK && L <= kLanesMaxL;
}

int batch_lanes_words(int L)
{
    const int Lh = (L + 1) / 2;
    return Lh <= 4 ? 4 : Lh <= 8 ? 8 : Lh <= 12 ? 12 : 16;
}

cudaError_t launch_batch_prep(int64_t B, int L, int k, const uint64_t *bits, const uint64_t *mem,
                              const uint64_t *cap, const uint32_t *bw, const BatchLanes &t, cudaStream_t s)
{
    if (B <= 0) return cudaSuccess;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int64_t blocks = (B + kPrepWarps - 1) / kPrepWarps;
    if (blocks > (int64_t)sms * 16) blocks = (int64_t)sms * 16;
    const int ufull = k * (k - 1), uhalf = ufull / 2;
    for (int pass = 0; pass < 2; ++pass) {
        const int ucap = pass ? ufull : uhalf;
        const size_t sm = prep_layout(L, ucap).total * kPrepWarps;
        // the attribute is set to the larger size both times: it belongs to the function, and another
        // host thread may be between its own two launches
        cudaError_t e = cudaFuncSetAttribute(k_lanes_prep, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)(prep_layout(L, ufull).total * kPrepWarps));
        if (e != cudaSuccess) return e;
        k_lanes_prep<<<(unsigned)blocks, kPrepWarps * 32, sm, s>>>(t, B, L, k, bits, mem, cap, bw, ucap, pass);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_batch_lanes(int64_t B, int L, int k, const uint64_t *bits, const uint32_t *bw,
                               const BatchLanes &t, double *beta, int32_t *m, int32_t *cuts,
                               int32_t *placement, int8_t *status, cudaStream_t s)
{
    if (B <= 0) return cudaSuccess;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t G = (B + 31) >> 5;
    const int jmax = k < L ? k : L;
    uint64_t binom = (uint64_t)k;  // C(k, j - 1), the source masks of level j
    const int64_t slots = (int64_t)sms * 16;  // warps the GPU holds at a time, roughly
    for (int j = 2; j <= jmax; ++j) {
        int split = 1;  // warps per source mask: a level with few masks spreads the k - j + 1 targets
        while (split < k - j + 1 && G * (int64_t)binom * split < 3 * slots) ++split;
        const int64_t items = G * (int64_t)binom * split;
        int64_t blocks = (items + kLevelWarps - 1) / kLevelWarps;
        const int64_t cap = (int64_t)sms * 32;
        if (blocks > cap) blocks = cap;
        cudaError_t e;
        switch (t.LH) {
            case 4: e = launch_level<4>(j - 1, t, B, k, L, split, (unsigned)blocks, s); break;
            case 8: e = launch_level<8>(j - 1, t, B, k, L, split, (unsigned)blocks, s); break;
            case 12: e = launch_level<12>(j - 1, t, B, k, L, split, (unsigned)blocks, s); break;
            case 16: e = launch_level<16>(j - 1, t, B, k, L, split, (unsigned)blocks, s); break;
            default: e = cudaErrorInvalidValue;
        }
        if (e != cudaSuccess) return e;
        binom = binom * (uint64_t)(k - j + 1) / (uint64_t)j;
    }
    int64_t blocks = (B + kBackWarps - 1) / kBackWarps;
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    return launch_dependent(k_lanes_back, (unsigned)blocks, kBackWarps * 32, 0, s, t, B, L, k, bits, bw, beta, m, cuts,
                            placement, status);
}

}  // namespace pp
