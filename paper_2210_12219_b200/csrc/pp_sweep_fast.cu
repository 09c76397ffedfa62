// Register-tiled sweep of one popcount level for 16-bit ranks.
//
// Envelope: 16-bit state elements, Lpad <= 240 (rows occupy at most 30 lanes) and the whole rank
// table in shared memory.  Two window steps: one for nodes whose sliding window has a constant
// width, lo_w(c') = max(0, c' - W_w), W_w >= 8 (chains whose layers all need the same memory,
// e.g. stacks of identical blocks), and one for arbitrary window tables that looks everything up
// in per-warp shared-memory strips.  Anything else runs on the generic kernel.
//
// Mapping: one warp per source mask S.  Lane l owns the 8 consecutive cut positions 8l..8l+7 of
// every row, as four packed u16x2 registers (one 16-byte vector).  The |S| source rows
// dp[S][v][.] are loaded once into registers; then, for every target node w not in S, the warp
//   1. relaxes   g[c] = min_v max(dp[S][v][c], rank[w][v][c])    (one 128-bit shared-memory load
//      and eight packed min/max per (v, w) and lane; two source nodes share a three-input min),
//   2. takes the window minimum  out[c'] = min g[c'-W .. c'-1]   with blocks of 8 = lanes:
//      window = tail of the block that holds c'-W  (in-lane suffix minima, published to a
//               per-warp strip and read back at offset -W)
//             + whole blocks in between            (sliding minimum over the block minima,
//               by doubling shuffles)
//             + head of the own block              (in-lane exclusive prefix minima),
//      all of it branch-free: what a node does not need is a shuffle from distance 31, which
//      finds no source lane and leaves the accumulator alone, or a read of the +inf pad,
//   3. writes row dp[S + w][w][.] with one 16-byte store per lane.
// The relaxation of the next target node is issued in the same straight-line block as the window
// step of the current one, so that independent loads fill the latencies of the dependent chain.
// Row (S + w, w) has the single source mask S, so no two warps ever write the same row.
#include <algorithm>

#include "pp_internal.cuh"
#include "pp_sweep_ops.cuh"

namespace pp {

namespace {

// Threads per block by the number of source rows a warp keeps in registers: fewer rows leave room
// for more resident warps (the register file holds 64K registers per SM).
constexpr int kMaxFastThreads = 768;
constexpr int kFastNv768 = 6, kFastNv640 = 9;  // 768 threads up to NV = 6, 640 up to 9, 512 above
__host__ __device__ constexpr int fast_threads(int nv, bool gen) { return gen ? 512 : (nv <= kFastNv768 ? 768 : (nv <= kFastNv640 ? 640 : 512)); }
// Per-target-node constants of the window step (W = 8q + r), built on the host.
// A shuffle distance of 31 means "nothing": rows occupy at most 30 lanes, so no lane that holds
// data finds a source and +inf (or the untouched accumulator) results.
struct alignas(16) WMeta {
    int toff;        // -ceil(W / 2): 32-bit word offset of position c' - W in the suffix strip
    int sh16;        // 16 if W is odd else 0
    int d1, d2;      // T1 = min(D << d1, D << d2): 1 and 1 + n1 - 2^s, or 31 when n1 = q - 1 = 0
    int dd[4];       // doubling distances 1, 2, 4, 8 for the first s steps, then 31
    int dq;          // q: the one more block that positions below r need
    int pad[3];
    uint32_t sel[4]; // byte selectors that pick T(q) or T(q-1) per half of each register
};

struct FastMeta {
    WMeta w[PP_MAX_K];
};

constexpr int NT = 1;  // target nodes processed together
// Per-warp strip of the general window step: the levels of the sparse table, then one word of +inf.
// A level is four planes of 32 words: plane i holds, for every lane, the lane's register i (cut
// positions 8 lane + 2 i and + 2 i + 1).  Position c of level s is therefore the halfword at
// gen_strip_byte(s, c): lanes that look up neighbouring positions hit neighbouring banks.
__host__ __device__ constexpr int gen_strip_elems(int levels, int /*Lpad*/) { return (levels * 128 + 4) * 2; }
__host__ __device__ constexpr uint32_t gen_strip_byte(int s, int c)
{
    return (uint32_t)((((s * 4 + ((c & 7) >> 1)) * 32 + (c >> 3)) << 2) + ((c & 1) << 1));
}
constexpr int kTailWords = 128 + 128;           // per-warp suffix strip of the constant-window step: +inf pad, data

// Window minimum of NT rows held as r[t][0..3]; result in o[t][0..3].  tl points at this lane's four
// words of the warp's suffix strip; the 128 words below the strip hold +inf.
__device__ __forceinline__ void window_min(const uint32_t (&r)[NT][4], const WMeta *const *mptr, uint32_t *tl,
                                           uint32_t (&o)[NT][4])
{
    static_assert(NT == 1, "the suffix strip holds one row at a time");
    // the constants of each node arrive as four 16-byte shared-memory loads
    union MetaRegs {
        WMeta m;
        uint4 q[sizeof(WMeta) / 16];
    };
    MetaRegs mr[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int i = 0; i < (int)(sizeof(WMeta) / 16); ++i)
            mr[t].q[i] = reinterpret_cast<const uint4 *>(mptr[t])[i];
    const WMeta *mp[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) mp[t] = &mr[t].m;
    uint32_t B[NT];
    uint32_t f[NT][5];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
        // pair minima replicated in both halves, their prefix (q*) and suffix (t*) minima
        const uint32_t m0 = vmin2(r[t][0], __byte_perm(r[t][0], 0, 0x1032));
        const uint32_t m1 = vmin2(r[t][1], __byte_perm(r[t][1], 0, 0x1032));
        const uint32_t m2 = vmin2(r[t][2], __byte_perm(r[t][2], 0, 0x1032));
        const uint32_t m3 = vmin2(r[t][3], __byte_perm(r[t][3], 0, 0x1032));
        const uint32_t q1 = vmin2(m0, m1), q2 = vmin2(q1, m2);
        const uint32_t t2 = vmin2(m2, m3), t1 = vmin2(m1, t2);
        B[t] = vmin2(q2, m3);
        // exclusive in-lane prefix minima: (min g[0..2j-1], min g[0..2j])
        o[t][0] = __byte_perm(r[t][0], kInf2, 0x1044);
        o[t][1] = vmin2(m0, __byte_perm(r[t][1], kInf2, 0x1044));
        o[t][2] = vmin2(q1, __byte_perm(r[t][2], kInf2, 0x1044));
        o[t][3] = vmin2(q2, __byte_perm(r[t][3], kInf2, 0x1044));
        // inclusive in-lane suffix minima: (min g[2j..7], min g[2j+1..7]), published to the strip
        const uint32_t s0 = vmin2(__byte_perm(m0, r[t][0], 0x7610), t1);
        const uint32_t s1 = vmin2(__byte_perm(m1, r[t][1], 0x7610), t2);
        const uint32_t s2 = vmin2(__byte_perm(m2, r[t][2], 0x7610), m3);
        const uint32_t s3 = __byte_perm(m3, r[t][3], 0x7610);
        __syncwarp();  // the previous row's readers are done
        *reinterpret_cast<uint4 *>(tl) = make_uint4(s0, s1, s2, s3);
        __syncwarp();
        // tail of the block that holds c' - W: the five words that cover positions c' - W of this
        // lane's eight outputs (negative positions read the +inf pad)
        const uint32_t *tp = tl + mp[t]->toff;
#pragma unroll
        for (int j = 0; j < 5; ++j) f[t][j] = tp[j];
    }
    // whole blocks in between: D = min B[l-2^s+1 .. l], T1 = min B[l-n1 .. l-1], T2 = min B[l-q .. l-1]
    uint32_t D[NT], T1[NT], T2[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) D[t] = B[t];
#pragma unroll
    for (int st = 0; st < 4; ++st)
#pragma unroll
        for (int t = 0; t < NT; ++t) min_shfl_up(D[t], D[t], mp[t]->dd[st]);
#pragma unroll
    for (int t = 0; t < NT; ++t) T1[t] = shfl_up_inf(D[t], mp[t]->d1);
#pragma unroll
    for (int t = 0; t < NT; ++t) min_shfl_up(T1[t], D[t], mp[t]->d2);
#pragma unroll
    for (int t = 0; t < NT; ++t) {
        T2[t] = T1[t];
        min_shfl_up(T2[t], B[t], mp[t]->dq);
    }
#pragma unroll
    for (int t = 0; t < NT; ++t) {
        const int sh = mp[t]->sh16;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            // an odd W straddles two words per output register
            const uint32_t e = __funnelshift_r(f[t][j], f[t][j + 1], sh);
            const uint32_t mid = __byte_perm(T2[t], T1[t], mp[t]->sel[j]);
            o[t][j] = vmin3(o[t][j], e, mid);
        }
    }
}

// Window minimum for arbitrary window starts lo_w(c'): a sparse table over the positions of the
// relaxed row, T[s][c] = min g[c - 2^s + 1 .. c], built in registers level by level (shifts by 1, 2
// and 4 positions inside a lane's 16-byte vector with one to two registers from the lane below,
// shifts by 8 and more as whole-lane shuffles) and parked in the warp's strip of shared memory.
// Output c' is then min(T[s][c' - 1], T[s][lo + 2^s - 1]) with 2^s <= c' - lo < 2^(s+1): two 16-bit
// loads whose byte offsets come from the lookup word the host prepared for (w, c')
// (gen_meta_build); an empty window points both at the +inf element behind the last level.
// Entries that would reach below position 0 hold garbage and are never asked for.
__device__ __forceinline__ void window_min_general(const uint32_t (&r)[4], const uint32_t *meta_row, uint16_t *T,
                                                   int lane, bool active, int nlev, int Lpad, uint32_t (&o)[4])
{
    uint32_t t[4] = {r[0], r[1], r[2], r[3]};
    uint32_t *mine = reinterpret_cast<uint32_t *>(T) + lane;  // this lane's word of plane 0, level 0
    auto park = [&](int s) {
        if (active) {
#pragma unroll
            for (int i = 0; i < 4; ++i) mine[(s * 4 + i) * 32] = t[i];
        }
    };
    __syncwarp();  // the previous row's readers are done with the strip
    park(0);
    if (nlev > 1) {  // shift by one position
        const uint32_t below = __shfl_up_sync(0xFFFFFFFFu, t[3], 1);
        const uint32_t y0 = __byte_perm(below, t[0], 0x5432), y1 = __byte_perm(t[0], t[1], 0x5432);
        const uint32_t y2 = __byte_perm(t[1], t[2], 0x5432), y3 = __byte_perm(t[2], t[3], 0x5432);
        t[0] = vmin2(t[0], y0); t[1] = vmin2(t[1], y1); t[2] = vmin2(t[2], y2); t[3] = vmin2(t[3], y3);
        park(1);
    }
    if (nlev > 2) {  // by two positions: one register
        const uint32_t below = __shfl_up_sync(0xFFFFFFFFu, t[3], 1);
        const uint32_t a0 = vmin2(t[0], below), a1 = vmin2(t[1], t[0]), a2 = vmin2(t[2], t[1]), a3 = vmin2(t[3], t[2]);
        t[0] = a0; t[1] = a1; t[2] = a2; t[3] = a3;
        park(2);
    }
    if (nlev > 3) {  // by four positions: two registers
        const uint32_t b2 = __shfl_up_sync(0xFFFFFFFFu, t[2], 1), b3 = __shfl_up_sync(0xFFFFFFFFu, t[3], 1);
        const uint32_t a0 = vmin2(t[0], b2), a1 = vmin2(t[1], b3), a2 = vmin2(t[2], t[0]), a3 = vmin2(t[3], t[1]);
        t[0] = a0; t[1] = a1; t[2] = a2; t[3] = a3;
        park(3);
    }
    for (int s = 4; s < nlev; ++s) {  // by 8 * 2^(s-4) positions: whole lanes
        const int dl = 1 << (s - 4);
#pragma unroll
        for (int j = 0; j < 4; ++j) t[j] = vmin2(t[j], __shfl_up_sync(0xFFFFFFFFu, t[j], dl));
        park(s);
    }
    __syncwarp();
    // lanes beyond the row take empty windows
    const uint32_t none = (uint32_t)(nlev * 128 * 4) * 0x10001u;
    const uint4 ma = active ? *reinterpret_cast<const uint4 *>(meta_row + 8 * lane) : make_uint4(none, none, none, none);
    const uint4 mb = active ? *reinterpret_cast<const uint4 *>(meta_row + 8 * lane + 4) : make_uint4(none, none, none, none);
    const uint32_t mw[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
    const unsigned char *Tb = reinterpret_cast<const unsigned char *>(T);
    uint32_t val[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t x = *reinterpret_cast<const uint16_t *>(Tb + (mw[i] & 0xFFFFu));
        const uint32_t y = *reinterpret_cast<const uint16_t *>(Tb + (mw[i] >> 16));
        val[i] = min(x, y);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) o[j] = val[2 * j] | (val[2 * j + 1] << 16);
}

template <int NV, bool GEN>
__global__ void __launch_bounds__(fast_threads(NV, GEN), 1)
k_sweep_fast(Dev d, int level, const FastMeta *__restrict__ meta_g, int split, int first_level)
{
    constexpr int kFastThreads = fast_threads(NV, GEN);
    // The first level of a solve follows the kernel that writes the rank table and the base
    // frontier: nothing may be read before that kernel is complete.
    if (first_level) asm volatile("griddepcontrol.wait;" ::: "memory");
    // Programmatic dependent launch: let the next level's blocks be scheduled as soon as this
    // level's blocks retire, so that their prologue (rank table -> shared memory) overlaps our
    // tail.  Nothing the previous level wrote is touched before griddepcontrol.wait below.
    asm volatile("griddepcontrol.launch_dependents;");
    extern __shared__ uint4 smem4[];
    uint16_t *rank_s = reinterpret_cast<uint16_t *>(smem4);
    const int k = d.k, L = d.L, Lpad = d.Lpad;
    const int rank_elems = k * k * Lpad;
    // table, then 512 bytes of slack for lanes beyond the row, then the per-node constants
    WMeta *wm = reinterpret_cast<WMeta *>(reinterpret_cast<unsigned char *>(smem4) +
                                          (((size_t)rank_elems * 2 + 512 + 15) & ~(size_t)15));
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(d.rank);
        for (int i = threadIdx.x; i < rank_elems / 8; i += kFastThreads) smem4[i] = src[i];
        for (int i = threadIdx.x; i < 32; i += kFastThreads)
            smem4[rank_elems / 8 + i] = make_uint4(kInf2, kInf2, kInf2, kInf2);
        if (!GEN) {
            const int *ms = reinterpret_cast<const int *>(meta_g);
            int *md = reinterpret_cast<int *>(wm);
            for (int i = threadIdx.x; i < (int)(sizeof(WMeta) / 4) * k; i += kFastThreads) md[i] = ms[i];
        }
    }
    // general windows: the lookup words of every (node, position) and three strips per warp live
    // behind the per-node constants
    uint32_t *gm_s = reinterpret_cast<uint32_t *>(wm + PP_MAX_K);
    // constant windows: per-warp suffix strip (128 words of +inf, then the row's 128 words)
    uint32_t *tl = gm_s + (threadIdx.x >> 5) * kTailWords + 128 + 4 * (threadIdx.x & 31);
    if (!GEN) {
        uint32_t *pad = gm_s + (threadIdx.x >> 5) * kTailWords;
        for (int i = threadIdx.x & 31; i < kTailWords; i += 32) pad[i] = kInf2;
    }
    uint16_t *strips = reinterpret_cast<uint16_t *>(gm_s + k * Lpad) +
                       (threadIdx.x >> 5) * gen_strip_elems(d.gen_levels, Lpad);
    if (GEN) {
        for (int i = threadIdx.x; i < k * Lpad; i += kFastThreads) gm_s[i] = d.gen_meta[i];
        if ((threadIdx.x & 31) == 0)  // the constant +inf behind the table
            *reinterpret_cast<uint32_t *>(strips + d.gen_levels * 256) = kInf2;
    }
    __syncthreads();
    if (!first_level) asm volatile("griddepcontrol.wait;" ::: "memory");  // previous level complete and visible

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nl = Lpad >> 3;  // lanes that hold a piece of a row
    const bool active = lane < nl;
    const uint16_t *table = reinterpret_cast<const uint16_t *>(d.table);
    uint16_t *table_w = reinterpret_cast<uint16_t *>(d.table);
    const uint32_t first = d.level_off[level - 1];
    // Work items: (mask, part).  Levels with few masks split each mask's target nodes over
    // `split` warps (part p takes the targets whose ordinal is p mod split), so that small
    // levels are not serialised on a handful of warps.
    const uint32_t nmask = (d.level_off[level] - first) * (uint32_t)split;
    const uint32_t full = (1u << k) - 1u;
    const int last_lane = (L - 1) >> 3, last_reg = ((L - 1) & 7) >> 1, last_sh = ((L - 1) & 1) * 16;
    const uint32_t stride = gridDim.x * (kFastThreads / 32);

    uint32_t mi = warp * gridDim.x + blockIdx.x;  // items go round the blocks: a partial last round spreads over all SMs
    uint32_t S = mi < nmask ? d.masks[first + mi / split] : 0u;
    int voff[NV];
    uint4 dp[NV];
    // best final key seen so far: read once per mask, not once per row (a stale value only costs a
    // redundant atomic); the read for the next mask is issued early and consumed after the last
    // row of the current one
    unsigned long long best_seen = kNoBest, best_next = kNoBest;
    // source rows of mask Sx -> registers
    auto load_rows = [&](uint32_t Sx) {
        uint32_t rem = Sx;
#pragma unroll
        for (int vi = 0; vi < NV; ++vi) {
            int v = __ffs(rem) - 1;
            rem &= rem - 1;
            voff[vi] = v * Lpad;
        }
        const uint16_t *src = table + (size_t)Sx * k * Lpad + 8 * lane;
#pragma unroll
        for (int vi = 0; vi < NV; ++vi)
            dp[vi] = active && PP_IN_BOUNDS(d, (size_t)Sx * k * Lpad + 8 * lane + voff[vi], d.table_elems)
                         ? __ldg(reinterpret_cast<const uint4 *>(src + voff[vi]))
                            : make_uint4(kInf2, kInf2, kInf2, kInf2);
        best_next = *reinterpret_cast<volatile unsigned long long *>(d.best);
    };
    if (mi < nmask) load_rows(S);
    best_seen = best_next;
    while (mi < nmask) {
        const uint32_t mi_next = mi + stride;
        const uint32_t S_next = mi_next < nmask ? d.masks[first + mi_next / split] : 0u;
        const uint32_t S_cur = S;
        uint32_t wrem = full & ~S_cur;
        uint16_t *const row_base = table_w + (size_t)S_cur * k * Lpad + 8 * lane;
        if (split > 1) {  // keep this part's share of the target nodes
            const int part = (int)(mi % (uint32_t)split);
            uint32_t keep = 0;
            int idx = 0;
            for (uint32_t rem = wrem; rem; rem &= rem - 1, ++idx)
                if (idx % split == part) keep |= rem & (0u - rem);
            wrem = keep;
        }
        const int npairs = (__popc(wrem) + NT - 1) / NT;  // target nodes of this item, NT at a time

        // next two target nodes (an odd tail repeats its last node), branch-free
        auto pick = [&](int (&w)[NT]) {
            w[0] = __ffs(wrem) - 1;
            wrem &= wrem - 1;
#pragma unroll
            for (int t = 1; t < NT; ++t) {
                w[t] = wrem ? __ffs(wrem) - 1 : w[t - 1];
                wrem &= wrem - 1;
            }
        };
        // 1. relax over the source nodes, two of them per three-input minimum
        auto relax = [&](const int (&w)[NT], uint32_t (&r)[NT][4]) {
            const uint16_t *rw[NT];
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                rw[t] = rank_s + w[t] * k * Lpad + 8 * lane;
                r[t][0] = r[t][1] = r[t][2] = r[t][3] = kInf2;
            }
#pragma unroll
            for (int vi = 0; vi + 1 < NV; vi += 2) {
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    const uint4 g = *reinterpret_cast<const uint4 *>(rw[t] + voff[vi]);
                    const uint4 h = *reinterpret_cast<const uint4 *>(rw[t] + voff[vi + 1]);
                    r[t][0] = vmin3(r[t][0], vmax2(dp[vi].x, g.x), vmax2(dp[vi + 1].x, h.x));
                    r[t][1] = vmin3(r[t][1], vmax2(dp[vi].y, g.y), vmax2(dp[vi + 1].y, h.y));
                    r[t][2] = vmin3(r[t][2], vmax2(dp[vi].z, g.z), vmax2(dp[vi + 1].z, h.z));
                    r[t][3] = vmin3(r[t][3], vmax2(dp[vi].w, g.w), vmax2(dp[vi + 1].w, h.w));
                }
            }
            if (NV & 1) {
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    const uint4 g = *reinterpret_cast<const uint4 *>(rw[t] + voff[NV - 1]);
                    r[t][0] = vmin2(r[t][0], vmax2(dp[NV - 1].x, g.x));
                    r[t][1] = vmin2(r[t][1], vmax2(dp[NV - 1].y, g.y));
                    r[t][2] = vmin2(r[t][2], vmax2(dp[NV - 1].z, g.z));
                    r[t][3] = vmin2(r[t][3], vmax2(dp[NV - 1].w, g.w));
                }
            }
        };
        // 2. + 3. window minimum, write the rows, offer their last elements as final states
        auto finish = [&](const int (&w)[NT], const uint32_t (&r)[NT][4]) {
            const WMeta *mp[NT];
#pragma unroll
            for (int t = 0; t < NT; ++t) mp[t] = wm + w[t];
            uint32_t o[NT][4];
            if (GEN)
                window_min_general(r[0], gm_s + w[0] * Lpad, strips, lane, active, d.gen_levels, Lpad, o[0]);
            else
                window_min(r, mp, tl, o);
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                const uint32_t S2 = S_cur | (1u << w[t]);
                if (active && PP_IN_BOUNDS(d, (size_t)S_cur * k * Lpad + 8 * lane + (size_t)((k << w[t]) + w[t]) * Lpad,
                                           d.table_elems))  // row (S2, w) lies ((k << w) + w) rows after row (S_cur, 0)
                    *reinterpret_cast<uint4 *>(row_base + (uint32_t)(((k << w[t]) + w[t]) * Lpad)) =
                        make_uint4(o[t][0], o[t][1], o[t][2], o[t][3]);
                const uint32_t reg = last_reg == 0 ? o[t][0] : (last_reg == 1 ? o[t][1] : (last_reg == 2 ? o[t][2] : o[t][3]));
                const uint32_t val = (reg >> last_sh) & 0xFFFFu;
                // ranks at or below the best rank seen so far are rare: everything else ends here
                if (lane == last_lane && val <= (uint32_t)(best_seen >> 30) && val != 0xFFFFu)
                    best_seen = offer_final(d.best, best_seen, val, level, S2, w[t]);
            }
        };
        // software pipeline over the pairs of target nodes: the relaxation of the next pair
        // (independent loads and min/max) sits in the same straight-line block as the window
        // step of the current pair (dependent shuffle chains), so the scheduler can fill the
        // latencies of one with the other
        int w[NT];
        uint32_t r[NT][4];
        pick(w);
        relax(w, r);
        for (int it = 1; it < npairs; ++it) {
            int wn[NT];
            uint32_t rn[NT][4];
            pick(wn);
            relax(wn, rn);
            finish(w, r);
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                w[t] = wn[t];
#pragma unroll
                for (int j = 0; j < 4; ++j) r[t][j] = rn[t][j];
            }
        }
        // the source rows are dead once the last pair is relaxed: fetch the next mask's rows now,
        // so that their latency hides behind the last window step
        if (mi_next < nmask) load_rows(S_next);
        finish(w, r);
        best_seen = best_next < best_seen ? best_next : best_seen;
        mi = mi_next;
        S = S_next;
    }
}

size_t fast_smem_bytes(const Dev &d)
{
    size_t b = (((size_t)d.k * d.k * d.Lpad * 2 + 512 + 15) & ~(size_t)15) + sizeof(WMeta) * PP_MAX_K;
    if (!d.fast_meta)  // general windows: lookup words + strips
        b += (size_t)d.k * d.Lpad * 4 + (size_t)(512 / 32) * gen_strip_elems(d.gen_levels, d.Lpad) * 2;
    else               // constant windows: suffix strips
        b += (size_t)(kMaxFastThreads / 32) * kTailWords * 4;
    return b;
}

template <int NV, bool GEN>
cudaError_t launch_nv(const Dev &d, int level, const FastMeta *meta, unsigned grid, int split, size_t sm, cudaStream_t s,
                      int first_level)
{
    cudaError_t e = cudaFuncSetAttribute(k_sweep_fast<NV, GEN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(fast_threads(NV, GEN));
    cfg.dynamicSmemBytes = sm;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_sweep_fast<NV, GEN>, d, level, meta, split, first_level);
}

}  // namespace

size_t fast_meta_bytes() { return sizeof(FastMeta); }

// Fills the per-node window constants; returns false when some node's window is not a constant
// width >= 8 (then the generic kernel must be used).  lo is the host window table [k*L].
bool fast_meta_build(int L, int k, const int16_t *lo, void *out)
{
    FastMeta *fm = static_cast<FastMeta *>(out);
    const int per32 = 16, Lpad = (L + per32 - 1) / per32 * per32;
    for (int w = 0; w < k; ++w) {
        int W = 0;
        for (int c2 = 0; c2 < L; ++c2) W = (c2 - lo[w * L + c2]) > W ? (c2 - lo[w * L + c2]) : W;
        for (int c2 = 0; c2 < L; ++c2)
            if (lo[w * L + c2] != (c2 - W > 0 ? c2 - W : 0)) return false;
        if (L > 1 && W < 8) return false;
        if (W >= L - 1) W = Lpad;  // the window always reaches layer 0: treat as "everything before"
        WMeta &m = fm->w[w];
        const int q = W >> 3, r = W & 7;
        auto clamp = [](int x) { return x > 31 ? 31 : x; };
        m.toff = -((W + 1) >> 1);
        m.sh16 = (r & 1) ? 16 : 0;
        const int n1 = q - 1 > 31 ? 31 : q - 1;
        int s = 0;
        while (n1 >= 1 && (2 << s) <= n1) ++s;
        for (int st = 0; st < 4; ++st) m.dd[st] = (n1 >= 1 && st < s) ? (1 << st) : 31;
        m.d1 = n1 >= 1 ? 1 : 31;
        m.d2 = n1 >= 1 ? 1 + n1 - (1 << s) : 31;
        m.dq = clamp(q);
        m.pad[0] = m.pad[1] = m.pad[2] = 0;
        for (int j = 0; j < 4; ++j)
            m.sel[j] = ((2 * j < r) ? 0x0010u : 0x0054u) | ((2 * j + 1 < r) ? 0x3200u : 0x7600u);
    }
    return true;
}

// Lookup words of the general window step (see window_min_general), row stride Lpad <= 240:
// byte offsets into a warp's strip of T[s][c' - 1] (low half) and T[s][lo + 2^s - 1] (high half),
// both the +inf element for an empty window.  Returns the number of table levels in use.
int gen_meta_build(int L, int k, int Lpad, const int16_t *lo, uint32_t *out)
{
    int maxlen = 1;
    for (int w = 0; w < k; ++w)
        for (int c2 = 0; c2 < L; ++c2) maxlen = std::max(maxlen, c2 - (int)lo[w * L + c2]);
    int levels = 1;
    while ((1 << levels) <= maxlen) ++levels;  // floor(log2(maxlen)) + 1
    const uint32_t inf_off = (uint32_t)(levels * 128 * 4);
    for (int w = 0; w < k; ++w)
        for (int c2 = 0; c2 < Lpad; ++c2) {
            const int a = c2 < L ? lo[w * L + c2] : c2;  // pads: empty window
            const int len = c2 - a;
            uint32_t o1 = inf_off, o2 = inf_off;
            if (len > 0) {
                int s = 0;
                while ((2 << s) <= len) ++s;
                o1 = gen_strip_byte(s, c2 - 1);
                o2 = gen_strip_byte(s, a + (1 << s) - 1);
            }
            out[w * Lpad + c2] = o1 | (o2 << 16);
        }
    return levels;
}

bool fast_sweep_supported(const Dev &d)
{
    if (d.elem != 2 || d.Lpad > 240 || d.k < 2 || d.k > PP_MAX_K || (!d.fast_meta && !d.gen_meta)) return false;
    int dev = 0, max_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&max_sm, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
    return fast_smem_bytes(d) <= (size_t)max_sm;
}

cudaError_t launch_sweep_fast(const Dev &d, int level, cudaStream_t s, bool first_level)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    unsigned long long n = 1;  // source masks of popcount level-1
    for (int i = 0; i < level - 1; ++i) n = n * (unsigned)(d.k - i) / (unsigned)(i + 1);
    const unsigned wpb = fast_threads(level - 1, d.fast_meta == nullptr) / 32;
    const int nw = d.k - (level - 1);  // target nodes per mask
    int split = 1;
    if (n < (unsigned long long)sms * wpb) {
        split = (int)(((unsigned long long)sms * wpb + n - 1) / n);
        if (split > nw) split = nw;
    }
    unsigned grid = (unsigned)((n * split + wpb - 1) / wpb);
    if (grid > (unsigned)sms) grid = (unsigned)sms;
    const size_t sm = fast_smem_bytes(d);
    const FastMeta *meta = static_cast<const FastMeta *>(d.fast_meta);
    switch (level - 1) {
#define PP_CASE(N) \
    case N: return meta ? launch_nv<N, false>(d, level, meta, grid, split, sm, s, first_level) \
                        : launch_nv<N, true>(d, level, meta, grid, split, sm, s, first_level);
        PP_CASE(1) PP_CASE(2) PP_CASE(3) PP_CASE(4) PP_CASE(5) PP_CASE(6) PP_CASE(7) PP_CASE(8)
        PP_CASE(9) PP_CASE(10) PP_CASE(11) PP_CASE(12) PP_CASE(13) PP_CASE(14) PP_CASE(15)
        PP_CASE(16) PP_CASE(17) PP_CASE(18) PP_CASE(19)
#undef PP_CASE
    }
    return cudaErrorInvalidValue;
}

}  // namespace pp
