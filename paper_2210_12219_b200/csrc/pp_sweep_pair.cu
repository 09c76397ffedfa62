// Register-tiled sweep of one popcount level, two source masks per warp.
//
// Same envelope as the constant-window variant of the one-mask kernel (16-bit ranks, Lpad <= 240,
// every node's window lo_w(c') = max(0, c' - W_w) with W_w >= 8, rank table in shared memory).
// The masks of a level are listed in revolving-door order, so masks 2i and 2i+1 differ by one swap:
// S1 = T + a, S2 = T + b.  A warp takes such a pair and keeps both sets of source rows in
// registers (lane l owns cut positions 8l..8l+7 of every row).  For every target node w outside T
//   1. both rows g1 = min_{v in S1} max(dp[S1][v], rank[w][v]),  g2 = the same over S2, are relaxed
//      together: the rank rows of the common sources T are read from shared memory once for the two
//      masks;
//   2. the two rows are re-packed position by position, (g1[c], g2[c]) in one register, so that the
//      window minimum runs on both at once: in-lane prefix / suffix minima need no permutes, and
//      the shuffles over block minima and the strip traffic are shared;
//   3. rows dp[S1 + w][w] and dp[S2 + w][w] are written (w = b only for S1, w = a only for S2).
// Window decomposition as in the one-mask kernel, blocks of 8 = lanes, W = 8q + r:
//   out[8l + j] = min( suffix of block l - q (j >= r) or l - q - 1 (j < r) from offset (j - r) mod 8,
//                      q - 1 (resp. q) whole blocks in between, prefix of the own block ).
// The suffix minima travel through a per-warp strip of 16 slots x 64 words.  Slots 8..15 hold the
// in-lane suffix minima sfx_i (i = slot - 8) of lane x at word 31 + x; slots 1..7 hold
// E_i = min(sfx_i, block minimum of the next lane) (i = slot), i.e. the suffix run on through one
// more block, at word 32 + x (word 31, the lane before lane 0, holds the minimum of block 0: its own
// suffixes are empty).  Output j then reads slot j - r + 8 at word 31 + l - q whatever j is:
// for j >= r that is sfx_{j-r} of lane l - q, for j < r it is E_{8+j-r} of lane l - q - 1, and in both
// cases the q - 1 whole blocks l-q+1 .. l-1 remain.  The words below 31 stay +inf.  Addresses
// differ by constants, nothing is selected, the code is branch-free, no access has a bank conflict.
#include "pp_internal.cuh"
#include "pp_sweep_ops.cuh"

namespace pp {

namespace {

// Tunables (measured on the k = 18, L = 200 benchmark chain): levels the kernel takes by number of
// source nodes, how full the machine must be (pairs * kPairFill >= warps), and threads per block by
// the number of source rows per mask (2 * NV rows of 4 registers per lane).
constexpr int kPairMinNv = 3, kPairMaxNv = 12;
constexpr int kPairT512 = 6, kPairT384 = 11;  // 512 threads up to NV = 6, 384 up to 11, 256 above
constexpr int kPairFill = 2;
__host__ __device__ constexpr int pair_threads(int nv) { return nv <= kPairT512 ? 512 : (nv <= kPairT384 ? 384 : 256); }
constexpr int kPlane = 64;               // words per strip slot
constexpr int kStripWords = 16 * kPlane;  // per warp
constexpr int kPlanWords = 32;            // per warp: row offsets of the pair to come

// Per-target-node constants (W = 8q + r), built on the host.  A shuffle distance of 31 means
// "nothing": rows occupy at most 30 lanes.
struct alignas(16) PMeta {
    int dd[4];   // doubling distances 1, 2, 4, 8 for the first s steps (2^s <= q - 1 < 2^(s+1)), then 31
    int d1, d2;  // T1 = min(D << d1, D << d2): 1 and q - 2^s, or 31 when q = 1
    int soff;    // (8 - r) * 64 - q: word offset from a lane's word of slot 0 to what its output 0 reads
    int rowoff;  // ((k << w) + w) * Lpad / 8: row (S + w, w) in 16-byte pieces after row (S, 0)
    int rwoff;   // w * k * Lpad: element offset of the node's block of the rank table
    int pad[3];
};

struct PairMeta {
    PMeta w[PP_MAX_K];
};

// 16-byte store under a predicate, no branch
__device__ __forceinline__ void st_if(uint4 *ptr, const uint4 &v, bool on)
{
    asm volatile("{ .reg .pred p; setp.ne.u32 p, %5, 0; @p st.global.v4.u32 [%0], {%1, %2, %3, %4}; }" ::"l"(ptr),
                 "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"((uint32_t)on)
                 : "memory");
}

__device__ __forceinline__ uint4 max4(const uint4 &a, const uint4 &b)
{
    return make_uint4(vmax2(a.x, b.x), vmax2(a.y, b.y), vmax2(a.z, b.z), vmax2(a.w, b.w));
}
__device__ __forceinline__ void set4(uint32_t (&r)[4], const uint4 &a)
{
    r[0] = a.x; r[1] = a.y; r[2] = a.z; r[3] = a.w;
}
__device__ __forceinline__ void min4(uint32_t (&r)[4], const uint4 &a)
{
    r[0] = vmin2(r[0], a.x); r[1] = vmin2(r[1], a.y); r[2] = vmin2(r[2], a.z); r[3] = vmin2(r[3], a.w);
}
__device__ __forceinline__ void min4(uint32_t (&r)[4], const uint4 &a, const uint4 &b)
{
    r[0] = vmin3(r[0], a.x, b.x); r[1] = vmin3(r[1], a.y, b.y);
    r[2] = vmin3(r[2], a.z, b.z); r[3] = vmin3(r[3], a.w, b.w);
}
__device__ __forceinline__ void setmin4(uint32_t (&r)[4], const uint4 &a, const uint4 &b, const uint4 &c)
{
    r[0] = vmin3(a.x, b.x, c.x); r[1] = vmin3(a.y, b.y, c.y); r[2] = vmin3(a.z, b.z, c.z); r[3] = vmin3(a.w, b.w, c.w);
}
__device__ __forceinline__ void setmin4(uint32_t (&r)[4], const uint4 &a, const uint4 &b)
{
    r[0] = vmin2(a.x, b.x); r[1] = vmin2(a.y, b.y); r[2] = vmin2(a.z, b.z); r[3] = vmin2(a.w, b.w);
}

// (t + 1, t + 1) for the best final rank t seen so far: a packed value x holds a rank <= t in
// one of its halves exactly when max(x, that) != x
__device__ __forceinline__ uint32_t offer_threshold(unsigned long long best_seen)
{
    const unsigned long long r = best_seen >> 30;
    const uint32_t t = (r > 0xFFFEull ? 0xFFFEu : (uint32_t)r) + 1u;
    return t | (t << 16);
}
// Slow path of the final-state bookkeeping for the two rows of a pair (x = their last elements).
__device__ __noinline__ unsigned long long offer_pair(unsigned long long *best, unsigned long long best_seen,
                                                      uint32_t x, bool ok1, bool ok2, int level, uint32_t A,
                                                      uint32_t B, int w)
{
    const uint32_t v1 = x & 0xFFFFu, v2 = x >> 16;
    if (ok1 && v1 != 0xFFFFu) best_seen = offer_final(best, best_seen, v1, level, A | (1u << w), w);
    if (ok2 && v2 != 0xFFFFu) best_seen = offer_final(best, best_seen, v2, level, B | (1u << w), w);
    return best_seen;
}


// L8: the chain length is a multiple of 8, so the last element of a row is a lane's last position.
template <int NV, bool L8>
__global__ void __launch_bounds__(pair_threads(NV), 1)
k_sweep_pair(Dev d, int level, const PairMeta *__restrict__ meta_g, int first_level)
{
    constexpr int kThreads = pair_threads(NV);
    constexpr int kWarps = kThreads / 32;
    constexpr int NC = NV - 1;  // sources common to both masks
    // The first level of a solve follows the kernel that writes the rank table and the base
    // frontier: nothing may be read before that kernel is complete.
    if (first_level) asm volatile("griddepcontrol.wait;" ::: "memory");
    // the next level's prologue (rank table -> shared memory) may overlap this level's tail
    asm volatile("griddepcontrol.launch_dependents;");
    extern __shared__ uint4 smem4[];
    uint16_t *rank_s = reinterpret_cast<uint16_t *>(smem4);
    const int k = d.k, L = d.L, Lpad = d.Lpad;
    const int rank_elems = k * k * Lpad;
    // table, 512 bytes of +inf for the lanes beyond the row, per-node constants, strips
    PMeta *wm = reinterpret_cast<PMeta *>(reinterpret_cast<unsigned char *>(smem4) +
                                          (((size_t)rank_elems * 2 + 512 + 15) & ~(size_t)15));
    uint32_t *strips = reinterpret_cast<uint32_t *>(wm + PP_MAX_K);
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(d.rank);
        for (int i = threadIdx.x; i < rank_elems / 8; i += kThreads) smem4[i] = src[i];
        for (int i = threadIdx.x; i < 32; i += kThreads)
            smem4[rank_elems / 8 + i] = make_uint4(kInf2, kInf2, kInf2, kInf2);
        const int *ms = reinterpret_cast<const int *>(meta_g);
        int *md = reinterpret_cast<int *>(wm);
        for (int i = threadIdx.x; i < (int)(sizeof(PMeta) / 4) * k; i += kThreads) md[i] = ms[i];
        for (int i = threadIdx.x; i < kWarps * kStripWords; i += kThreads) strips[i] = kInf2;
    }
    __syncthreads();
    if (!first_level) asm volatile("griddepcontrol.wait;" ::: "memory");  // previous level complete and visible

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int l8 = Lpad >> 3;  // 16-byte pieces per row
    const bool active = lane < l8;
    uint32_t *const sl = strips + warp * kStripWords + 31 + lane;  // this lane's word of slot 0
    int *const wo = reinterpret_cast<int *>(strips + kWarps * kStripWords) + warp * kPlanWords;  // row offsets of a pair
    uint32_t *const se = strips + warp * kStripWords + (lane == 31 ? 31 : 32 + lane);  // ... of the E slots
    const int next_lane = (lane + 1) & 31;
    // rows are addressed in 16-byte pieces from the start of the table (fits 32 bits at every size)
    const uint4 *const table = reinterpret_cast<const uint4 *>(d.table);
    uint4 *const table_w = reinterpret_cast<uint4 *>(d.table);
    const uint32_t first = d.level_off[level - 1];
    const uint32_t nmask = d.level_off[level] - first;
    const uint32_t npair = (nmask + 1) >> 1;
    const uint32_t full = (1u << k) - 1u;
    const bool is_last = lane == ((L - 1) >> 3);
    const int last_j = (L - 1) & 7;
    const uint32_t stride = gridDim.x * kWarps;
    const uint4 inf4 = make_uint4(kInf2, kInf2, kInf2, kInf2);
    const uint32_t mask_rows = (uint32_t)(k * l8);  // pieces per mask

    // pair p goes to block p mod gridDim (round by round over the warp slots): the last, partial
    // round is then spread over all SMs instead of filling a few of them
    uint32_t pi = warp * gridDim.x + blockIdx.x;
    // sources: voff[0 .. NV-2] the common nodes T, voff[NV-1] = a (S1 only), voffb = b (S2 only);
    // offsets in elements from the start of a rank-table block or a mask's rows
    int voff[NV];
    int voffb = 0;
    uint4 dp1[NV], dp2[NV];
    unsigned long long best_seen = kNoBest, best_next = kNoBest;
    uint32_t S1 = 0, S2 = 0;
    auto fetch_masks = [&](uint32_t p, uint32_t &A, uint32_t &B) {
        A = d.masks[first + 2 * p];
        B = (2 * p + 1 < nmask) ? d.masks[first + 2 * p + 1] : A;
    };
    // Rows of the pair (A, B).  plan_rows works out where they are (in 16-byte pieces from the first
    // row of a mask) once, leaves the offsets in the warp's scratch words, and starts the rows on
    // their way into L2 (one 16-byte piece per lane covers a row); load_rows1 / load_rows2 fetch the
    // rows of A / of B into the registers later, and load_rows2 takes over the pair's source offsets.
    auto plan_rows = [&](uint32_t A, uint32_t B, bool prefetch) {
        uint32_t abit = A & ~B;
        if (!abit) abit = A & (0u - A);  // a mask without partner runs as a pair with itself
        const uint32_t T = A & ~abit;
        const uint32_t bbit = B & ~T;
        const uint32_t i1 = A * mask_rows + lane, i2 = B * mask_rows + lane;
        uint32_t rem = T;
        __syncwarp();  // the previous plan has been read
#pragma unroll
        for (int vi = 0; vi <= NV; ++vi) {
            const uint32_t bits = vi < NC ? rem : (vi == NC ? abit : bbit);
            const int off = (__ffs(bits) - 1) * l8;
            if (vi < NC) rem &= rem - 1;
            wo[vi] = off;
            if (prefetch && active) {
                if (vi < NV) asm volatile("prefetch.global.L2 [%0];" ::"l"(table + (i1 + off)));
                if (vi != NC) asm volatile("prefetch.global.L2 [%0];" ::"l"(table + (i2 + off)));
            }
        }
        __syncwarp();
    };
    auto load_rows1 = [&](uint32_t A) {
        const uint32_t i1 = A * mask_rows + lane;
#pragma unroll
        for (int vi = 0; vi < NV; ++vi)
            dp1[vi] = active && PP_IN_BOUNDS(d, (uint64_t)(i1 + wo[vi]) * 8, d.table_elems) ? __ldg(table + (i1 + wo[vi])) : inf4;
    };
    auto load_rows2 = [&](uint32_t B) {
        const uint32_t i2 = B * mask_rows + lane;
#pragma unroll
        for (int vi = 0; vi < NV; ++vi) {
            voff[vi] = wo[vi] * 8;
            const uint32_t at = i2 + wo[vi == NC ? NV : vi];
            dp2[vi] = active && PP_IN_BOUNDS(d, (uint64_t)at * 8, d.table_elems) ? __ldg(table + at) : inf4;
        }
        voffb = wo[NV] * 8;
        best_next = *reinterpret_cast<volatile unsigned long long *>(d.best);
    };
    // the masks of a pair are fetched two pairs ahead: their latency never meets a dependent instruction
    uint32_t S1n = 0, S2n = 0;
    if (pi < npair) {
        fetch_masks(pi, S1, S2);
        if (pi + stride < npair) fetch_masks(pi + stride, S1n, S2n);
        plan_rows(S1, S2, false);
        load_rows1(S1);
        load_rows2(S2);
    }
    best_seen = best_next;
    uint32_t thr2 = offer_threshold(best_seen);
    while (pi < npair) {
        const uint32_t pi_next = pi + stride;
        const bool more = pi_next < npair;
        uint32_t S1nn = 0, S2nn = 0;
        if (pi_next + stride < npair) fetch_masks(pi_next + stride, S1nn, S2nn);
        const uint32_t A = S1, B = S2;
        const uint32_t base1 = A * mask_rows + lane, base2 = B * mask_rows + lane;

        // 1. both rows relaxed over their sources, two sources per three-input minimum
        auto relax = [&](int w, uint32_t (&r1)[4], uint32_t (&r2)[4]) {
            const uint16_t *rw = rank_s + wm[w].rwoff + 8 * lane;
            const uint4 ga = *reinterpret_cast<const uint4 *>(rw + voff[NV - 1]);
            const uint4 gb = *reinterpret_cast<const uint4 *>(rw + voffb);
            if (NC >= 2) {
                // the first minimum takes three sources (two common ones and the mask's own), every
                // further one two more: ceil((NV - 1) / 2) three-input minima per register
                const uint4 g = *reinterpret_cast<const uint4 *>(rw + voff[0]);
                const uint4 h = *reinterpret_cast<const uint4 *>(rw + voff[NC >= 2 ? 1 : 0]);
                setmin4(r1, max4(dp1[0], g), max4(dp1[NC >= 2 ? 1 : 0], h), max4(dp1[NV - 1], ga));
                setmin4(r2, max4(dp2[0], g), max4(dp2[NC >= 2 ? 1 : 0], h), max4(dp2[NV - 1], gb));
#pragma unroll
                for (int vi = 2; vi + 1 < NC; vi += 2) {
                    const uint4 g2 = *reinterpret_cast<const uint4 *>(rw + voff[vi]);
                    const uint4 h2 = *reinterpret_cast<const uint4 *>(rw + voff[vi + 1]);
                    min4(r1, max4(dp1[vi], g2), max4(dp1[vi + 1], h2));
                    min4(r2, max4(dp2[vi], g2), max4(dp2[vi + 1], h2));
                }
                if (NC & 1) {  // one common source is left over
                    const uint4 g3 = *reinterpret_cast<const uint4 *>(rw + voff[NC - 1]);
                    min4(r1, max4(dp1[NC - 1], g3));
                    min4(r2, max4(dp2[NC - 1], g3));
                }
            } else if (NC == 1) {
                const uint4 g = *reinterpret_cast<const uint4 *>(rw + voff[0]);
                setmin4(r1, max4(dp1[0], g), max4(dp1[NV - 1], ga));
                setmin4(r2, max4(dp2[0], g), max4(dp2[NV - 1], gb));
            } else {
                set4(r1, max4(dp1[NV - 1], ga));
                set4(r2, max4(dp2[NV - 1], gb));
            }
        };
        // one row only (the target is a node of the other mask): sources T and `lastoff`
        auto relax1 = [&](int w, const uint4 (&dp)[NV], int lastoff, uint32_t (&r)[4]) {
            const uint16_t *rw = rank_s + wm[w].rwoff + 8 * lane;
            const uint4 ga = *reinterpret_cast<const uint4 *>(rw + lastoff);
            if (NC >= 2) {
                const uint4 g = *reinterpret_cast<const uint4 *>(rw + voff[0]);
                const uint4 h = *reinterpret_cast<const uint4 *>(rw + voff[NC >= 2 ? 1 : 0]);
                setmin4(r, max4(dp[0], g), max4(dp[NC >= 2 ? 1 : 0], h), max4(dp[NV - 1], ga));
#pragma unroll
                for (int vi = 2; vi + 1 < NC; vi += 2) {
                    const uint4 g2 = *reinterpret_cast<const uint4 *>(rw + voff[vi]);
                    const uint4 h2 = *reinterpret_cast<const uint4 *>(rw + voff[vi + 1]);
                    min4(r, max4(dp[vi], g2), max4(dp[vi + 1], h2));
                }
                if (NC & 1) {
                    const uint4 g3 = *reinterpret_cast<const uint4 *>(rw + voff[NC >= 1 ? NC - 1 : 0]);
                    min4(r, max4(dp[NC >= 1 ? NC - 1 : 0], g3));
                }
            } else if (NC == 1) {
                const uint4 g = *reinterpret_cast<const uint4 *>(rw + voff[0]);
                setmin4(r, max4(dp[0], g), max4(dp[NV - 1], ga));
            } else {
                set4(r, max4(dp[NV - 1], ga));
            }
        };
        // 2. + 3. window minimum of both rows, write them, offer their last elements as final states
        auto finish = [&](int w, const uint32_t (&r1)[4], const uint32_t (&r2)[4], bool ok1, bool ok2) {
            const uint4 ma = *reinterpret_cast<const uint4 *>(&wm[w].dd[0]);
            const uint4 mb = *reinterpret_cast<const uint4 *>(&wm[w].d1);  // d1, d2, soff, rowoff
            // p[j] = (g1[8l + j], g2[8l + j])
            uint32_t p[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                p[2 * j] = __byte_perm(r1[j], r2[j], 0x5410);
                p[2 * j + 1] = __byte_perm(r1[j], r2[j], 0x7632);
            }
            // in-lane inclusive suffix minima s[j] = min p[j..7], exclusive prefix minima o[j] = min p[0..j-1]
            uint32_t s[8], o[8];
            s[7] = p[7];
#pragma unroll
            for (int j = 6; j >= 0; --j) s[j] = vmin2(p[j], s[j + 1]);
            o[0] = kInf2;
            o[1] = p[0];
#pragma unroll
            for (int j = 2; j < 8; ++j) o[j] = vmin2(o[j - 1], p[j - 1]);
            // E_i = min(s_i, block minimum of the next lane).  Lane 31 never holds a piece of a row
            // (its s_i are +inf); it takes the block minimum of lane 0 and writes the entries of the
            // lane "before lane 0", whose suffixes are empty but whose next block is block 0.
            const uint32_t Bn = __shfl_sync(0xFFFFFFFFu, s[0], next_lane);
            // whole blocks in between: D = min B[l-2^s+1 .. l], T1 = min B[l-q+1 .. l-1].  A lane without
            // a source lane gets its own value back from the shuffle, which leaves D alone.  The chain of
            // dependent shuffles is spread over the strip traffic below.
            uint32_t D = s[0];
            D = vmin2(D, __shfl_up_sync(0xFFFFFFFFu, D, ma.x));
            __syncwarp();  // the previous rows' readers are done
#pragma unroll
            for (int j = 0; j < 8; ++j) sl[(8 + j) * kPlane] = s[j];
            D = vmin2(D, __shfl_up_sync(0xFFFFFFFFu, D, ma.y));
#pragma unroll
            for (int j = 1; j < 8; ++j) se[j * kPlane] = vmin2(s[j], Bn);
            D = vmin2(D, __shfl_up_sync(0xFFFFFFFFu, D, ma.z));
            __syncwarp();
            const uint32_t *sp = sl + (int)mb.z;
            uint32_t f[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) f[j] = sp[j * kPlane];
            D = vmin2(D, __shfl_up_sync(0xFFFFFFFFu, D, ma.w));
            const uint32_t T1 = vmin2(shfl_up_inf(D, (int)mb.x), shfl_up_inf(D, (int)mb.y));
            uint32_t out[8];
            out[0] = vmin2(f[0], T1);
#pragma unroll
            for (int j = 1; j < 8; ++j) out[j] = vmin3(o[j], f[j], T1);
            // row (S + w, w) lies rowoff pieces after row (S, 0)
            if (ok1)
                st_if(table_w + (base1 + mb.w),
                      make_uint4(__byte_perm(out[0], out[1], 0x5410), __byte_perm(out[2], out[3], 0x5410),
                                 __byte_perm(out[4], out[5], 0x5410), __byte_perm(out[6], out[7], 0x5410)),
                      active && PP_IN_BOUNDS(d, (uint64_t)(base1 + mb.w) * 8, d.table_elems));
            if (ok2)
                st_if(table_w + (base2 + mb.w),
                      make_uint4(__byte_perm(out[0], out[1], 0x7632), __byte_perm(out[2], out[3], 0x7632),
                                 __byte_perm(out[4], out[5], 0x7632), __byte_perm(out[6], out[7], 0x7632)),
                      active && PP_IN_BOUNDS(d, (uint64_t)(base2 + mb.w) * 8, d.table_elems));
            // final states: ranks at or below the best rank seen so far are rare
            uint32_t x = out[7];
            if (!L8) {
                const uint32_t x01 = (last_j & 1) ? out[1] : out[0], x23 = (last_j & 1) ? out[3] : out[2];
                const uint32_t x45 = (last_j & 1) ? out[5] : out[4], x67 = (last_j & 1) ? out[7] : out[6];
                const uint32_t x03 = (last_j & 2) ? x23 : x01, x47 = (last_j & 2) ? x67 : x45;
                x = (last_j & 4) ? x47 : x03;
            }
            if (is_last && vmax2(x, thr2) != x) {
                best_seen = offer_pair(d.best, best_seen, x, ok1, ok2, level, A, B, w);
                thr2 = offer_threshold(best_seen);
            }
        };
        uint32_t r1[4], r2[4];
        if (A != B) {
            const uint32_t abit = A & ~B, bbit = B & ~A;
            // targets outside both masks: two rows each
            uint32_t wrem = full & ~(A | B);
            // rows of the next pair on their way into L2 while this pair is worked on
            if (more) plan_rows(S1n, S2n, true);
            while (wrem) {
                const int w = __ffs(wrem) - 1;
                wrem &= wrem - 1;
                relax(w, r1, r2);
                finish(w, r1, r2, true, true);
            }
            // target b takes the rows of S1 only, target a those of S2; once a mask's rows are dead
            // the next pair's rows are fetched into their registers, behind the remaining window steps
            {
                const int w = __ffs(bbit) - 1;
                relax1(w, dp1, voff[NV - 1], r1);
                if (more) load_rows1(S1n);
                finish(w, r1, r1, true, false);
            }
            {
                const int w = __ffs(abit) - 1;
                relax1(w, dp2, voffb, r2);
                if (more) load_rows2(S2n);
                finish(w, r2, r2, false, true);
            }
        } else {
            // a mask without partner: one row per target
            uint32_t wrem = full & ~A;
            if (more) plan_rows(S1n, S2n, true);
            while (wrem) {
                const int w = __ffs(wrem) - 1;
                wrem &= wrem - 1;
                relax1(w, dp1, voff[NV - 1], r1);
                finish(w, r1, r1, true, false);
            }
            if (more) {
                load_rows1(S1n);
                load_rows2(S2n);
            }
        }
        if (best_next < best_seen) {
            best_seen = best_next;
            thr2 = offer_threshold(best_seen);
        }
        pi = pi_next;
        S1 = S1n;
        S2 = S2n;
        S1n = S1nn;
        S2n = S2nn;
    }
}

size_t pair_smem_bytes(const Dev &d, int nv)
{
    return (((size_t)d.k * d.k * d.Lpad * 2 + 512 + 15) & ~(size_t)15) + sizeof(PMeta) * PP_MAX_K +
           (size_t)(pair_threads(nv) / 32) * (kStripWords + kPlanWords) * 4;
}

template <int NV, bool L8>
cudaError_t launch_pair_nv(const Dev &d, int level, unsigned grid, size_t sm, cudaStream_t s, int first_level)
{
    cudaError_t e = cudaFuncSetAttribute(k_sweep_pair<NV, L8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(pair_threads(NV));
    cfg.dynamicSmemBytes = sm;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_sweep_pair<NV, L8>, d, level, static_cast<const PairMeta *>(d.pair_meta),
                              first_level);
}

}  // namespace

size_t pair_meta_bytes() { return sizeof(PairMeta); }

// Fills the per-node window constants; returns false when some node's window is not a constant
// width >= 8.  lo is the host window table [k*L].
bool pair_meta_build(int L, int k, const int16_t *lo, void *out)
{
    PairMeta *pm = static_cast<PairMeta *>(out);
    const int Lpad = (L + 15) / 16 * 16;
    for (int w = 0; w < k; ++w) {
        int W = 0;
        for (int c2 = 0; c2 < L; ++c2) W = (c2 - lo[w * L + c2]) > W ? (c2 - lo[w * L + c2]) : W;
        for (int c2 = 0; c2 < L; ++c2)
            if (lo[w * L + c2] != (c2 - W > 0 ? c2 - W : 0)) return false;
        if (L > 1 && W < 8) return false;
        if (W >= L - 1) W = Lpad;  // the window always reaches layer 0: treat as "everything before"
        PMeta &m = pm->w[w];
        const int q = W >> 3, r = W & 7;
        const int n1 = q - 1 > 31 ? 31 : q - 1;
        int s = 0;
        while (n1 >= 1 && (2 << s) <= n1) ++s;
        for (int st = 0; st < 4; ++st) m.dd[st] = (n1 >= 1 && st < s) ? (1 << st) : 31;
        m.d1 = n1 >= 1 ? 1 : 31;
        m.d2 = n1 >= 1 ? 1 + n1 - (1 << s) : 31;
        m.soff = (8 - r) * kPlane - q;
        m.rwoff = w * k * Lpad;
        m.rowoff = ((k << w) + w) * (Lpad / 8);
        m.pad[0] = m.pad[1] = m.pad[2] = 0;
    }
    return true;
}

// Levels the two-mask kernel takes: constant windows, masks in revolving-door order, enough
// source rows per mask to be worth sharing, few enough to fit the register file, and enough
// pairs to fill the machine (whenever_possible drops the last two: every level it can run).
bool pair_sweep_takes(const Dev &d, int level, bool whenever_possible)
{
    const int nv = level - 1;
    if (!d.pair_meta || d.elem != 2 || d.Lpad > 240) return false;
    if (whenever_possible ? (nv < 2 || nv > 13) : (nv < kPairMinNv || nv > kPairMaxNv)) return false;
    int dev = 0, max_sm = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&max_sm, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    if (pair_smem_bytes(d, nv) > (size_t)max_sm) return false;
    unsigned long long n = 1;  // source masks of popcount nv
    for (int i = 0; i < nv; ++i) n = n * (unsigned)(d.k - i) / (unsigned)(i + 1);
    return whenever_possible || (n + 1) / 2 * kPairFill >= (unsigned long long)sms * (pair_threads(nv) / 32);
}

cudaError_t launch_sweep_pair(const Dev &d, int level, cudaStream_t s, bool first_level)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int nv = level - 1;
    unsigned long long n = 1;
    for (int i = 0; i < nv; ++i) n = n * (unsigned)(d.k - i) / (unsigned)(i + 1);
    const unsigned wpb = pair_threads(nv) / 32;
    unsigned long long blocks = ((n + 1) / 2 + wpb - 1) / wpb;
    const unsigned grid = blocks > (unsigned long long)sms ? (unsigned)sms : (unsigned)blocks;
    const size_t sm = pair_smem_bytes(d, nv);
    switch (nv) {
#define PP_CASE(N) \
    case N: return (d.L & 7) ? launch_pair_nv<N, false>(d, level, grid, sm, s, first_level) \
                             : launch_pair_nv<N, true>(d, level, grid, sm, s, first_level);
        PP_CASE(2) PP_CASE(3) PP_CASE(4) PP_CASE(5) PP_CASE(6) PP_CASE(7) PP_CASE(8)
        PP_CASE(9) PP_CASE(10) PP_CASE(11) PP_CASE(12) PP_CASE(13)
#undef PP_CASE
    }
    return cudaErrorInvalidValue;
}

}  // namespace pp
