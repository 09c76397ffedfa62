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
//   1. k_batch in its preparing mode (pp_batch.cu), one block per instance: staging, windows, the
//      ranking of gamma (Eq. 3); writes the instance's column of the rank table, the window lengths,
//      the base frontier and the best single-node plan;
//   2. one launch per popcount level, k_lanes_level<NV, LH>: a warp takes (group of 32 instances,
//      source mask P of NV nodes), keeps the NV rows of P in registers (two cut positions per 32-bit
//      word, LH words per row), and for every node w outside P forms
//      g[c] = min_v max(dp[P][v][c], rank[v][w][c]) with packed 16-bit min/max, takes the window
//      minimum over [lo_w(c'), c'-1] (a fully unrolled scan over the distance, cut short at the
//      longest window of the warp, a lane's shorter window masked arithmetically), stores the row of (P + w, w), and keeps the smallest final state
//      (value, popcount, mask, node), merged into the instance's key with one atomic per lane;
//   3. k_lanes_back, one warp per instance: the value of the winning rank and the backtrack by the
//      threshold rule, lanes over the candidates.
// Same recurrence, final choice and backtrack rule as the single-instance path (pp_sweep.cu).
#include "pp_internal.cuh"

namespace pp {

namespace {

constexpr int kLevelWarps = 4;
constexpr int kBackWarps = 8;
constexpr int kLanesMinB = 64;  // below this the block-per-instance kernel keeps more of the GPU busy
constexpr int kLanesMaxK = 8;   // NV <= 7 rows of a source mask in registers
constexpr int kLanesMaxL = 32;  // LH <= 16 words per row
constexpr uint32_t kMagic = 0x4B000000u;     // bit pattern of 2^23: kMagic | r is the float 2^23 + r for r < 2^23
constexpr uint32_t kMagicInf = 0x4B00FFFFu;  // the rank of +inf in that form; also caps a masked candidate

template <int NV, int LH>
__global__ void __launch_bounds__(kLevelWarps * 32)
k_lanes_level(const BatchLanes t, const int64_t B, const int k, const int L)
{
    const int lane = threadIdx.x & 31;
    const uint32_t nmasks = t.moff[NV + 1] - t.moff[NV];
    const int64_t G = (B + 31) >> 5;
    const int64_t items = G * nmasks;
    const uint32_t full = (1u << k) - 1u;
    const int wfin = (L - 1) >> 1, sfin = ((L - 1) & 1) * 16;
    for (int64_t item = (int64_t)blockIdx.x * kLevelWarps + (threadIdx.x >> 5); item < items;
         item += (int64_t)gridDim.x * kLevelWarps) {
        const int64_t g = item / nmasks;
        const uint32_t P = t.mlist[t.moff[NV] + (uint32_t)(item - g * nmasks)];
        // lanes past the end of the batch read the last instance's column and store to their own
        const int64_t left = B - g * 32;
        const int valid = left < 32 ? (int)left : 32;
        const int col = lane < valid ? lane : valid - 1;
        const uint32_t *tab = t.table + (size_t)g * t.rows * (LH * 32) + col;
        uint32_t *tabw = t.table + (size_t)g * t.rows * (LH * 32) + lane;
        const uint32_t *rk = t.rank + (size_t)g * (size_t)(k * k) * (LH * 32) + col;
        const uint32_t *ln = t.len + (size_t)g * (size_t)k * (LH * 32) + col;
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
                for (int wd = 0; wd < LH; ++wd) d[vi][wd] = tab[((size_t)(row0 + vi) * LH + wd) * 32];
            }
        }
        unsigned long long key = kNoBest;
        for (uint32_t wrem = full & ~P; wrem; wrem &= wrem - 1) {
            const int w = __ffs(wrem) - 1;
            uint32_t gg[LH];
            {
                const uint32_t *r0 = rk + (size_t)((vs[0] * k + w) * LH) * 32;
#pragma unroll
                for (int wd = 0; wd < LH; ++wd) gg[wd] = __vmaxu2(d[0][wd], r0[wd * 32]);
            }
#pragma unroll
            for (int vi = 1; vi + 1 < NV; vi += 2) {
                const uint32_t *r1 = rk + (size_t)((vs[vi] * k + w) * LH) * 32;
                const uint32_t *r2 = rk + (size_t)((vs[vi + 1] * k + w) * LH) * 32;
#pragma unroll
                for (int wd = 0; wd < LH; ++wd)
                    gg[wd] = __vimin3_u16x2(gg[wd], __vmaxu2(d[vi][wd], r1[wd * 32]),
                                            __vmaxu2(d[vi + 1][wd], r2[wd * 32]));
            }
            if (!(NV & 1)) {
                const uint32_t *r1 = rk + (size_t)((vs[NV - 1] * k + w) * LH) * 32;
#pragma unroll
                for (int wd = 0; wd < LH; ++wd) gg[wd] = __vminu2(gg[wd], __vmaxu2(d[NV - 1][wd], r1[wd * 32]));
            }
            // window lengths of this node, and the longest one among the 32 instances
            uint32_t lw[LH];
            uint32_t m2 = 0;
#pragma unroll
            for (int wd = 0; wd < LH; ++wd) {
                lw[wd] = ln[(size_t)(w * LH + wd) * 32];
                m2 = __vmaxu2(m2, lw[wd]);
            }
            const int wmax = (int)__reduce_max_sync(0xFFFFFFFFu, max(m2 & 0xFFFFu, m2 >> 16));
            // The window minimum runs on floats that hold 2^23 + rank exactly (such floats order like
            // their bit patterns): out[c2] = min of g over the len(c2) positions before c2.  Every
            // distance up to the warp's longest window is taken; a lane whose own window is shorter
            // adds 2^16 to the candidate, t = saturate(distance - len) being 0 inside the window and
            // 1 outside, so that the masking is two multiply-add-pipe instructions and the 3-input
            // integer minimum takes two candidates at a time.
            float uf[2 * LH], lf[2 * LH];
#pragma unroll
            for (int wd = 0; wd < LH; ++wd) {
                uf[2 * wd] = __uint_as_float(__byte_perm(gg[wd], kMagic, 0x7610));
                uf[2 * wd + 1] = __uint_as_float(__byte_perm(gg[wd], kMagic, 0x7632));
                lf[2 * wd] = __uint_as_float(__byte_perm(lw[wd], kMagic, 0x7610));
                lf[2 * wd + 1] = __uint_as_float(__byte_perm(lw[wd], kMagic, 0x7632));
            }
            // distances in blocks of four, all positions inside a block: the positions are independent
            // of one another, and the test against the warp's longest window is made once per block
            int ob[2 * LH];
#pragma unroll
            for (int c2 = 0; c2 < 2 * LH; ++c2) ob[c2] = (int)kMagicInf;
#pragma unroll
            for (int d0 = 1; d0 < 2 * LH; d0 += 4) {
                if (d0 > wmax) break;
#pragma unroll
                for (int c2 = d0; c2 < 2 * LH; ++c2) {
                    int x[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int dd = d0 + q;
                        x[q] = (int)kMagicInf;
                        if (dd <= c2) {
                            const float t = __saturatef((8388608.0f + (float)dd) - lf[c2]);
                            x[q] = __float_as_int(fmaf(t, 65536.0f, uf[c2 - dd]));
                        }
                    }
                    ob[c2] = __vimin3_s32(ob[c2], x[0], x[1]);
                    if (d0 + 2 <= c2) ob[c2] = __vimin3_s32(ob[c2], x[2], x[3]);
                }
            }
            const uint32_t S2 = P | (1u << w);
            const uint32_t row = t.rowoff[S2] + (uint32_t)__popc(S2 & ((1u << w) - 1u));
            uint32_t xw = 0xFFFFFFFFu;
#pragma unroll
            for (int wd = 0; wd < LH; ++wd) {
                const uint32_t o = __byte_perm((uint32_t)ob[2 * wd], (uint32_t)ob[2 * wd + 1], 0x5410);
                tabw[((size_t)row * LH + wd) * 32] = o;
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
__device__ __forceinline__ uint32_t lanes_elem(const uint32_t *base, size_t row, int LH, int c)
{
    return (base[(row * LH + (size_t)(c >> 1)) * 32] >> ((c & 1) * 16)) & 0xFFFFu;
}

__global__ void __launch_bounds__(kBackWarps * 32)
k_lanes_back(const BatchLanes t, const int64_t B, const int L, const int k, const uint64_t *__restrict__ g_bits,
             const uint32_t *__restrict__ g_bw, double *__restrict__ o_beta, int32_t *__restrict__ o_m,
             int32_t *__restrict__ o_cuts, int32_t *__restrict__ o_place, int8_t *__restrict__ o_status)
{
    const int lane = threadIdx.x & 31;
    const int LH = t.LH;
    const double kInf = __longlong_as_double(0x7FF0000000000000ll);
    for (int64_t inst = (int64_t)blockIdx.x * kBackWarps + (threadIdx.x >> 5); inst < B;
         inst += (int64_t)gridDim.x * kBackWarps) {
        const size_t g = (size_t)(inst >> 5);
        const int col = (int)(inst & 31);
        const uint32_t *tab = t.table + g * t.rows * (size_t)(LH * 32) + col;
        const uint32_t *rk = t.rank + g * (size_t)(k * k) * (size_t)(LH * 32) + col;
        const uint32_t *ln = t.len + g * (size_t)k * (size_t)(LH * 32) + col;
        const unsigned long long key = t.key[inst];
        const int bad = t.flag[inst];
        int32_t *cuts = o_cuts ? o_cuts + inst * (k - 1) : nullptr;
        int32_t *place = o_place + inst * k;
        if (lane < k) place[lane] = -1;
        if (cuts && lane < k - 1) cuts[lane] = -1;
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
            for (int e = lane; e < k * k * LH; e += 32) {
                const uint32_t x = rk[(size_t)e * 32];
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
        }
        for (int j = m - 1; j >= 0; --j) {
            if (lane == 0) {
                place[j] = w;
                if (j < m - 1) cuts[j] = c2;
            }
            if (j == 0) break;
            const uint32_t P = S & ~(1u << w);
            const int l0 = c2 - (int)lanes_elem(ln, (size_t)w, LH, c2);
            const uint32_t prow = t.rowoff[P];
            unsigned int pick = 0xFFFFFFFFu;
            for (int base = 0; base < (c2 - l0) * k && pick == 0xFFFFFFFFu; base += 32) {
                const int it = base + lane;
                if (it < (c2 - l0) * k) {
                    const int c = l0 + it / k, v = it - (it / k) * k;
                    if ((P >> v) & 1u) {
                        const uint32_t a = lanes_elem(tab, (size_t)prow + __popc(P & ((1u << v) - 1u)), LH, c);
                        const uint32_t b = lanes_elem(rk, (size_t)(v * k + w), LH, c);
                        const uint32_t mx = a > b ? a : b;
                        if (mx <= rstar) pick = ((unsigned)c << 5) | (unsigned)v;
                    }
                }
                // candidates ascend with the lane (position first, then node): the first hit of the
                // earliest chunk that has one is the smallest (position, node)
                for (int o = 16; o; o >>= 1) {
                    const unsigned int other = __shfl_xor_sync(0xFFFFFFFFu, pick, o);
                    pick = other < pick ? other : pick;
                }
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

template <int LH>
cudaError_t launch_level(int nv, const BatchLanes &t, int64_t B, int k, int L, unsigned grid, cudaStream_t s)
{
    switch (nv) {
#define PP_CASE(N) \
    case N: k_lanes_level<N, LH><<<grid, kLevelWarps * 32, 0, s>>>(t, B, k, L); break;
        PP_CASE(1) PP_CASE(2) PP_CASE(3) PP_CASE(4) PP_CASE(5) PP_CASE(6) PP_CASE(7)
#undef PP_CASE
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
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
    for (int j = 2; j <= jmax; ++j) {
        const int64_t items = G * (int64_t)binom;
        int64_t blocks = (items + kLevelWarps - 1) / kLevelWarps;
        const int64_t cap = (int64_t)sms * 32;
        if (blocks > cap) blocks = cap;
        cudaError_t e;
        switch (t.LH) {
            case 4: e = launch_level<4>(j - 1, t, B, k, L, (unsigned)blocks, s); break;
            case 8: e = launch_level<8>(j - 1, t, B, k, L, (unsigned)blocks, s); break;
            case 12: e = launch_level<12>(j - 1, t, B, k, L, (unsigned)blocks, s); break;
            case 16: e = launch_level<16>(j - 1, t, B, k, L, (unsigned)blocks, s); break;
            default: e = cudaErrorInvalidValue;
        }
        if (e != cudaSuccess) return e;
        binom = binom * (uint64_t)(k - j + 1) / (uint64_t)j;
    }
    int64_t blocks = (B + kBackWarps - 1) / kBackWarps;
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    k_lanes_back<<<(unsigned)blocks, kBackWarps * 32, 0, s>>>(t, B, L, k, bits, bw, beta, m, cuts, placement, status);
    return cudaGetLastError();
}

}  // namespace pp
