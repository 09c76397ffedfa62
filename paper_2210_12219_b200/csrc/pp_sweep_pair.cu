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
//      window minimum runs on both at once: in-lane prefix / suffix minima need no permutes, the
//      shuffles over block minima and the strip traffic are shared, and the last combine is chosen
//      by a warp-uniform switch on W mod 8, which makes every register index static;
//   3. rows dp[S1 + w][w] and dp[S2 + w][w] are written (w = b only for S1, w = a only for S2).
// Window decomposition as in the one-mask kernel, blocks of 8 = lanes, W = 8q + r:
//   out[8l + j] = min( suffix of block l - q (j >= r) or l - q - 1 (j < r) from offset (j - r) mod 8,
//                      q - 1 (resp. q) whole blocks in between, prefix of the own block ).
// The suffix minima travel through a per-warp strip of 8 planes (one per offset) x 64 words
// (32 words of +inf, then one word per lane), so that all accesses are conflict-free.
#include "pp_internal.cuh"
#include "pp_sweep_ops.cuh"

namespace pp {

namespace {

#ifndef PP_PAIR_T512
#define PP_PAIR_T512 6
#endif
#ifndef PP_PAIR_MIN_NV
#define PP_PAIR_MIN_NV 3
#endif
#ifndef PP_PAIR_MAX_NV
#define PP_PAIR_MAX_NV 11
#endif
// threads per block by the number of source rows per mask (2 * NV rows of 4 registers per lane)
__host__ __device__ constexpr int pair_threads(int nv) { return nv <= PP_PAIR_T512 ? 512 : 384; }
constexpr int kMaxPairWarps = 16;
constexpr int kPlane = 64;              // words per strip plane
constexpr int kStripWords = 8 * kPlane;  // per warp

// Per-target-node constants (W = 8q + r), built on the host.  A shuffle distance of 31 means
// "nothing": rows occupy at most 30 lanes.
struct alignas(16) PMeta {
    int dd[4];   // doubling distances 1, 2, 4, 8 for the first s steps (2^s <= q - 1 < 2^(s+1)), then 31
    int d1, d2;  // T1 = min(D << d1, D << d2): 1 and q - 2^s, or 31 when q = 1
    int dq;      // q: the one more block that offsets below r need
    int qr;      // q | r << 8
};

struct PairMeta {
    PMeta w[PP_MAX_K];
};

// Last combine for W mod 8 == R.  sp = this lane's word of plane 0, moved back by q lanes.
template <int R>
__device__ __forceinline__ void pair_combine(const uint32_t *sp, const uint32_t (&o)[8], uint32_t T1, uint32_t T2,
                                             uint32_t (&out)[8])
{
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const uint32_t f = sp[((j - R) & 7) * kPlane - (j < R ? 1 : 0)];
        const uint32_t mid = j < R ? T2 : T1;
        out[j] = j == 0 ? vmin2(f, mid) : vmin3(o[j], f, mid);
    }
}

template <int NV>
__global__ void __launch_bounds__(pair_threads(NV), 1)
k_sweep_pair(Dev d, int level, const PairMeta *__restrict__ meta_g)
{
    constexpr int kThreads = pair_threads(NV);
    constexpr int kWarps = kThreads / 32;
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
    asm volatile("griddepcontrol.wait;" ::: "memory");  // previous level complete and visible

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const bool active = lane < (Lpad >> 3);
    uint32_t *const sl = strips + warp * kStripWords + 32 + lane;  // this lane's word of plane 0
    const uint16_t *table = reinterpret_cast<const uint16_t *>(d.table);
    uint16_t *table_w = reinterpret_cast<uint16_t *>(d.table);
    const uint32_t first = d.level_off[level - 1];
    const uint32_t nmask = d.level_off[level] - first;
    const uint32_t npair = (nmask + 1) >> 1;
    const uint32_t full = (1u << k) - 1u;
    const int last_lane = (L - 1) >> 3, last_j = (L - 1) & 7;
    const uint32_t stride = gridDim.x * kWarps;
    const uint4 inf4 = make_uint4(kInf2, kInf2, kInf2, kInf2);

    uint32_t pi = blockIdx.x * kWarps + warp;
    // sources: voff[0 .. NV-2] the common nodes T, voff[NV-1] = a (S1 only), voffb = b (S2 only)
    int voff[NV];
    int voffb = 0;
    uint4 dp1[NV], dp2[NV];
    unsigned long long best_seen = kNoBest, best_next = kNoBest;
    uint32_t S1 = 0, S2 = 0;
    auto fetch_masks = [&](uint32_t p, uint32_t &A, uint32_t &B) {
        A = d.masks[first + 2 * p];
        B = (2 * p + 1 < nmask) ? d.masks[first + 2 * p + 1] : A;
    };
    auto load_rows = [&](uint32_t A, uint32_t B) {
        uint32_t abit = A & ~B;
        if (!abit) abit = A & (0u - A);  // a mask without partner runs as a pair with itself
        const uint32_t T = A & ~abit;
        const uint32_t bbit = B & ~T;
        uint32_t rem = T;
#pragma unroll
        for (int vi = 0; vi < NV - 1; ++vi) {
            voff[vi] = (__ffs(rem) - 1) * Lpad;
            rem &= rem - 1;
        }
        voff[NV - 1] = (__ffs(abit) - 1) * Lpad;
        voffb = (__ffs(bbit) - 1) * Lpad;
        const uint16_t *s1 = table + (size_t)A * k * Lpad + 8 * lane;
        const uint16_t *s2 = table + (size_t)B * k * Lpad + 8 * lane;
#pragma unroll
        for (int vi = 0; vi < NV; ++vi) {
            dp1[vi] = active ? __ldg(reinterpret_cast<const uint4 *>(s1 + voff[vi])) : inf4;
            dp2[vi] = active ? __ldg(reinterpret_cast<const uint4 *>(s2 + (vi == NV - 1 ? voffb : voff[vi]))) : inf4;
        }
        best_next = *reinterpret_cast<volatile unsigned long long *>(d.best);
    };
    if (pi < npair) {
        fetch_masks(pi, S1, S2);
        load_rows(S1, S2);
    }
    best_seen = best_next;
    while (pi < npair) {
        const uint32_t pi_next = pi + stride;
        uint32_t S1n = 0, S2n = 0;
        if (pi_next < npair) fetch_masks(pi_next, S1n, S2n);
        const uint32_t A = S1, B = S2;
        const bool has2 = A != B;
        uint32_t wrem = full & ~(A & B);  // every node outside the common part
        uint16_t *const base1 = table_w + (size_t)A * k * Lpad + 8 * lane;
        uint16_t *const base2 = table_w + (size_t)B * k * Lpad + 8 * lane;
        const int ntargets = __popc(wrem);

        // 1. both rows relaxed over their sources, two sources per three-input minimum
        auto relax = [&](int w, uint32_t (&r1)[4], uint32_t (&r2)[4]) {
            const uint16_t *rw = rank_s + w * k * Lpad + 8 * lane;
#pragma unroll
            for (int j = 0; j < 4; ++j) r1[j] = r2[j] = kInf2;
#pragma unroll
            for (int vi = 0; vi + 1 < NV - 1; vi += 2) {
                const uint4 g = *reinterpret_cast<const uint4 *>(rw + voff[vi]);
                const uint4 h = *reinterpret_cast<const uint4 *>(rw + voff[vi + 1]);
                r1[0] = vmin3(r1[0], vmax2(dp1[vi].x, g.x), vmax2(dp1[vi + 1].x, h.x));
                r1[1] = vmin3(r1[1], vmax2(dp1[vi].y, g.y), vmax2(dp1[vi + 1].y, h.y));
                r1[2] = vmin3(r1[2], vmax2(dp1[vi].z, g.z), vmax2(dp1[vi + 1].z, h.z));
                r1[3] = vmin3(r1[3], vmax2(dp1[vi].w, g.w), vmax2(dp1[vi + 1].w, h.w));
                r2[0] = vmin3(r2[0], vmax2(dp2[vi].x, g.x), vmax2(dp2[vi + 1].x, h.x));
                r2[1] = vmin3(r2[1], vmax2(dp2[vi].y, g.y), vmax2(dp2[vi + 1].y, h.y));
                r2[2] = vmin3(r2[2], vmax2(dp2[vi].z, g.z), vmax2(dp2[vi + 1].z, h.z));
                r2[3] = vmin3(r2[3], vmax2(dp2[vi].w, g.w), vmax2(dp2[vi + 1].w, h.w));
            }
            const uint4 ga = *reinterpret_cast<const uint4 *>(rw + voff[NV - 1]);
            const uint4 gb = *reinterpret_cast<const uint4 *>(rw + voffb);
            if ((NV - 1) & 1) {  // the last common source shares a minimum with a (resp. b)
                const uint4 g = *reinterpret_cast<const uint4 *>(rw + voff[NV - 2 >= 0 ? NV - 2 : 0]);
                constexpr int c = NV - 2 >= 0 ? NV - 2 : 0;
                r1[0] = vmin3(r1[0], vmax2(dp1[c].x, g.x), vmax2(dp1[NV - 1].x, ga.x));
                r1[1] = vmin3(r1[1], vmax2(dp1[c].y, g.y), vmax2(dp1[NV - 1].y, ga.y));
                r1[2] = vmin3(r1[2], vmax2(dp1[c].z, g.z), vmax2(dp1[NV - 1].z, ga.z));
                r1[3] = vmin3(r1[3], vmax2(dp1[c].w, g.w), vmax2(dp1[NV - 1].w, ga.w));
                r2[0] = vmin3(r2[0], vmax2(dp2[c].x, g.x), vmax2(dp2[NV - 1].x, gb.x));
                r2[1] = vmin3(r2[1], vmax2(dp2[c].y, g.y), vmax2(dp2[NV - 1].y, gb.y));
                r2[2] = vmin3(r2[2], vmax2(dp2[c].z, g.z), vmax2(dp2[NV - 1].z, gb.z));
                r2[3] = vmin3(r2[3], vmax2(dp2[c].w, g.w), vmax2(dp2[NV - 1].w, gb.w));
            } else {
                r1[0] = vmin2(r1[0], vmax2(dp1[NV - 1].x, ga.x));
                r1[1] = vmin2(r1[1], vmax2(dp1[NV - 1].y, ga.y));
                r1[2] = vmin2(r1[2], vmax2(dp1[NV - 1].z, ga.z));
                r1[3] = vmin2(r1[3], vmax2(dp1[NV - 1].w, ga.w));
                r2[0] = vmin2(r2[0], vmax2(dp2[NV - 1].x, gb.x));
                r2[1] = vmin2(r2[1], vmax2(dp2[NV - 1].y, gb.y));
                r2[2] = vmin2(r2[2], vmax2(dp2[NV - 1].z, gb.z));
                r2[3] = vmin2(r2[3], vmax2(dp2[NV - 1].w, gb.w));
            }
        };
        // 2. + 3. window minimum of both rows, write them, offer their last elements as final states
        auto finish = [&](int w, const uint32_t (&r1)[4], const uint32_t (&r2)[4]) {
            const uint4 ma = *reinterpret_cast<const uint4 *>(&wm[w].dd[0]);
            const uint4 mb = *reinterpret_cast<const uint4 *>(&wm[w].d1);
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
            __syncwarp();  // the previous rows' readers are done
#pragma unroll
            for (int j = 0; j < 8; ++j) sl[j * kPlane] = s[j];
            __syncwarp();
            // whole blocks in between: D = min B[l-2^s+1 .. l], T1 = min B[l-q+1 .. l-1], T2 = min B[l-q .. l-1]
            uint32_t D = s[0];
            min_shfl_up(D, D, (int)ma.x);
            min_shfl_up(D, D, (int)ma.y);
            min_shfl_up(D, D, (int)ma.z);
            min_shfl_up(D, D, (int)ma.w);
            uint32_t T1 = shfl_up_inf(D, (int)mb.x);
            min_shfl_up(T1, D, (int)mb.y);
            uint32_t T2 = T1;
            min_shfl_up(T2, s[0], (int)mb.z);
            const int q = (int)(mb.w & 0xFFu), r = (int)(mb.w >> 8);
            const uint32_t *sp = sl - q;
            uint32_t out[8];
            switch (r) {
                case 0: pair_combine<0>(sp, o, T1, T2, out); break;
                case 1: pair_combine<1>(sp, o, T1, T2, out); break;
                case 2: pair_combine<2>(sp, o, T1, T2, out); break;
                case 3: pair_combine<3>(sp, o, T1, T2, out); break;
                case 4: pair_combine<4>(sp, o, T1, T2, out); break;
                case 5: pair_combine<5>(sp, o, T1, T2, out); break;
                case 6: pair_combine<6>(sp, o, T1, T2, out); break;
                default: pair_combine<7>(sp, o, T1, T2, out); break;
            }
            const bool ok1 = !((A >> w) & 1u), ok2 = has2 && !((B >> w) & 1u);
            const uint32_t rowoff = (uint32_t)(((k << w) + w) * Lpad);  // row (S + w, w) from row (S, 0)
            if (active && ok1)
                *reinterpret_cast<uint4 *>(base1 + rowoff) =
                    make_uint4(__byte_perm(out[0], out[1], 0x5410), __byte_perm(out[2], out[3], 0x5410),
                               __byte_perm(out[4], out[5], 0x5410), __byte_perm(out[6], out[7], 0x5410));
            if (active && ok2)
                *reinterpret_cast<uint4 *>(base2 + rowoff) =
                    make_uint4(__byte_perm(out[0], out[1], 0x7632), __byte_perm(out[2], out[3], 0x7632),
                               __byte_perm(out[4], out[5], 0x7632), __byte_perm(out[6], out[7], 0x7632));
            // final states: ranks at or below the best rank seen so far are rare
            uint32_t x;
            switch (last_j) {
                case 0: x = out[0]; break;
                case 1: x = out[1]; break;
                case 2: x = out[2]; break;
                case 3: x = out[3]; break;
                case 4: x = out[4]; break;
                case 5: x = out[5]; break;
                case 6: x = out[6]; break;
                default: x = out[7]; break;
            }
            const uint32_t v1 = ok1 ? (x & 0xFFFFu) : 0xFFFFu, v2 = ok2 ? (x >> 16) : 0xFFFFu;
            if (lane == last_lane && min(v1, v2) <= (uint32_t)(best_seen >> 30)) {
                if (v1 != 0xFFFFu && v1 <= (uint32_t)(best_seen >> 30))
                    best_seen = offer_final(d.best, best_seen, v1, level, A | (1u << w), w);
                if (v2 != 0xFFFFu && v2 <= (uint32_t)(best_seen >> 30))
                    best_seen = offer_final(d.best, best_seen, v2, level, B | (1u << w), w);
            }
        };
        // software pipeline over the target nodes: the relaxation of the next one (independent
        // loads and min/max) sits in the same straight-line block as the window step of the
        // current one (dependent shuffle chains)
        int w = __ffs(wrem) - 1;
        wrem &= wrem - 1;
        uint32_t r1[4], r2[4];
        relax(w, r1, r2);
        for (int it = 1; it < ntargets; ++it) {
            const int wn = __ffs(wrem) - 1;
            wrem &= wrem - 1;
            uint32_t rn1[4], rn2[4];
            relax(wn, rn1, rn2);
            finish(w, r1, r2);
            w = wn;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                r1[j] = rn1[j];
                r2[j] = rn2[j];
            }
        }
        // the source rows are dead once the last target is relaxed: fetch the next pair's rows
        // now, so that their latency hides behind the last window step
        if (pi_next < npair) load_rows(S1n, S2n);
        finish(w, r1, r2);
        best_seen = best_next < best_seen ? best_next : best_seen;
        pi = pi_next;
        S1 = S1n;
        S2 = S2n;
    }
}

size_t pair_smem_bytes(const Dev &d)
{
    return (((size_t)d.k * d.k * d.Lpad * 2 + 512 + 15) & ~(size_t)15) + sizeof(PMeta) * PP_MAX_K +
           (size_t)kMaxPairWarps * kStripWords * 4;
}

template <int NV>
cudaError_t launch_pair_nv(const Dev &d, int level, unsigned grid, size_t sm, cudaStream_t s)
{
    cudaError_t e = cudaFuncSetAttribute(k_sweep_pair<NV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
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
    return cudaLaunchKernelEx(&cfg, k_sweep_pair<NV>, d, level, static_cast<const PairMeta *>(d.pair_meta));
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
        m.dq = q > 31 ? 31 : q;
        m.qr = q | (r << 8);
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
    if (whenever_possible ? (nv < 2 || nv > 12) : (nv < PP_PAIR_MIN_NV || nv > PP_PAIR_MAX_NV)) return false;
    int dev = 0, max_sm = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&max_sm, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
    if (pair_smem_bytes(d) > (size_t)max_sm) return false;
    unsigned long long n = 1;  // source masks of popcount nv
    for (int i = 0; i < nv; ++i) n = n * (unsigned)(d.k - i) / (unsigned)(i + 1);
    return whenever_possible || (n + 1) / 2 >= (unsigned long long)sms * (pair_threads(nv) / 32);
}

cudaError_t launch_sweep_pair(const Dev &d, int level, cudaStream_t s)
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
    const size_t sm = pair_smem_bytes(d);
    switch (nv) {
#define PP_CASE(N) \
    case N: return launch_pair_nv<N>(d, level, grid, sm, s);
        PP_CASE(2) PP_CASE(3) PP_CASE(4) PP_CASE(5) PP_CASE(6) PP_CASE(7) PP_CASE(8)
        PP_CASE(9) PP_CASE(10) PP_CASE(11) PP_CASE(12)
#undef PP_CASE
    }
    return cudaErrorInvalidValue;
}

}  // namespace pp
