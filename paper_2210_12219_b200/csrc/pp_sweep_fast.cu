// Register-tiled sweep of one popcount level for 16-bit ranks.
//
// Envelope: 16-bit state elements, Lpad <= 256, the whole rank table in shared memory, and for
// every node w a sliding window of constant width:  lo_w(c') = max(0, c' - W_w), W_w >= 8 (chains
// whose layers all need the same memory, e.g. stacks of identical blocks).  Anything else runs on
// the generic kernel.
//
// Mapping: one warp per source mask S.  Lane l owns the 8 consecutive cut positions 8l..8l+7 of
// every row, as four packed u16x2 registers (one 16-byte vector).  The |S| source rows
// dp[S][v][.] are loaded once into registers; for every target node w not in S the warp
//   1. relaxes   g[c] = min_v max(dp[S][v][c], rank[w][v][c])    (one 128-bit shared-memory load
//      and eight packed min/max per (v, w) and lane),
//   2. takes the window minimum  out[c'] = min g[c'-W .. c'-1]   with blocks of 8 = lanes:
//      window = tail of the block that holds c'-W  (in-lane suffix minima, fetched by shuffles)
//             + whole blocks in between            (sliding minimum over the 32 block minima)
//             + head of the own block              (in-lane exclusive prefix minima),
//   3. writes row dp[S + w][w][.] with one 16-byte store per lane.
// Row (S + w, w) has the single source mask S, so no two warps ever write the same row.
#include "pp_internal.cuh"

namespace pp {

namespace {

constexpr int kFastThreads = 512;
constexpr uint32_t kInf2 = 0xFFFFFFFFu;

// per-target-node constants of the window step, precomputed on the host side of the launch
struct WMeta {
    int q, r;        // W = 8q + r
    int sh16;        // 16 if r is odd else 0
    int rr;          // r >> 1
    int jm;          // index of the register that mixes two source lanes (r odd), else -1
    int n1;          // q - 1: whole blocks between, for outputs at in-block positions >= r
    int s;           // floor(log2(n1)) when n1 >= 1
    int d2;          // 1 + n1 - 2^s
    uint32_t sel[4]; // byte selectors that pick T(q) or T(q-1) per half of each register
};

struct FastMeta {
    WMeta w[PP_MAX_K];
};

__device__ __forceinline__ uint32_t vmin2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("min.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t vmax2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
// shuffle up by delta lanes, +inf shifted in from below lane 0
__device__ __forceinline__ uint32_t shfl_up_inf(uint32_t x, int delta, int lane)
{
    uint32_t y = __shfl_up_sync(0xFFFFFFFFu, x, delta > 31 ? 31 : delta);
    return lane >= delta ? y : kInf2;
}

template <int NV>
__global__ void __launch_bounds__(kFastThreads, 1)
k_sweep_fast(Dev d, int level, const FastMeta *__restrict__ meta_g)
{
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
        for (int i = threadIdx.x; i < 32; i += kFastThreads) smem4[rank_elems / 8 + i] = make_uint4(kInf2, kInf2, kInf2, kInf2);
        const int *ms = reinterpret_cast<const int *>(meta_g);
        int *md = reinterpret_cast<int *>(wm);
        for (int i = threadIdx.x; i < (int)(sizeof(WMeta) / 4) * k; i += kFastThreads) md[i] = ms[i];
    }
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nl = Lpad >> 3;  // lanes that hold a piece of a row
    const bool active = lane < nl;
    const uint16_t *table = reinterpret_cast<const uint16_t *>(d.table);
    uint16_t *table_w = reinterpret_cast<uint16_t *>(d.table);
    const uint32_t first = d.level_off[level - 1];
    const uint32_t nmask = d.level_off[level] - first;
    const uint32_t full = (1u << k) - 1u;
    const int last_lane = (L - 1) >> 3, last_reg = ((L - 1) & 7) >> 1, last_half = (L - 1) & 1;

    for (uint32_t mi = blockIdx.x * (kFastThreads / 32) + warp; mi < nmask;
         mi += gridDim.x * (kFastThreads / 32)) {
        const uint32_t S = d.masks[first + mi];
        int voff[NV];
        uint4 dp[NV];
        {
            uint32_t rem = S;
#pragma unroll
            for (int vi = 0; vi < NV; ++vi) {
                int v = __ffs(rem) - 1;
                rem &= rem - 1;
                voff[vi] = v * Lpad;
            }
            const uint16_t *src = table + (size_t)S * k * Lpad + 8 * lane;
#pragma unroll
            for (int vi = 0; vi < NV; ++vi)
                dp[vi] = active ? __ldg(reinterpret_cast<const uint4 *>(src + voff[vi]))
                                : make_uint4(kInf2, kInf2, kInf2, kInf2);
        }
        for (uint32_t wrem = full & ~S; wrem; wrem &= wrem - 1) {
            const int w = __ffs(wrem) - 1;
            // ---- 1. relax over the source nodes ----
            const uint16_t *rw = rank_s + w * k * Lpad + 8 * lane;
            uint32_t r0 = kInf2, r1 = kInf2, r2 = kInf2, r3 = kInf2;
#pragma unroll
            for (int vi = 0; vi < NV; ++vi) {
                const uint4 g = *reinterpret_cast<const uint4 *>(rw + voff[vi]);
                r0 = vmin2(r0, vmax2(dp[vi].x, g.x));
                r1 = vmin2(r1, vmax2(dp[vi].y, g.y));
                r2 = vmin2(r2, vmax2(dp[vi].z, g.z));
                r3 = vmin2(r3, vmax2(dp[vi].w, g.w));
            }
            // ---- 2. window minimum ----
            const WMeta m = wm[w];
            // pair minima replicated in both halves, their prefix (q*) and suffix (t*) minima
            const uint32_t m0 = vmin2(r0, __byte_perm(r0, 0, 0x1032));
            const uint32_t m1 = vmin2(r1, __byte_perm(r1, 0, 0x1032));
            const uint32_t m2 = vmin2(r2, __byte_perm(r2, 0, 0x1032));
            const uint32_t m3 = vmin2(r3, __byte_perm(r3, 0, 0x1032));
            const uint32_t q1 = vmin2(m0, m1), q2 = vmin2(q1, m2), B = vmin2(q2, m3);
            const uint32_t t2 = vmin2(m2, m3), t1 = vmin2(m1, t2);
            // exclusive in-lane prefix minima: (min g[0..2j-1], min g[0..2j])
            uint32_t o0 = (r0 << 16) | 0xFFFFu;
            uint32_t o1 = vmin2(m0, (r1 << 16) | 0xFFFFu);
            uint32_t o2 = vmin2(q1, (r2 << 16) | 0xFFFFu);
            uint32_t o3 = vmin2(q2, (r3 << 16) | 0xFFFFu);
            // inclusive in-lane suffix minima: (min g[2j..7], min g[2j+1..7])
            uint32_t z0 = vmin2(__byte_perm(m0, r0, 0x7610), t1);
            uint32_t z1 = vmin2(__byte_perm(m1, r1, 0x7610), t2);
            uint32_t z2 = vmin2(__byte_perm(m2, r2, 0x7610), m3);
            uint32_t z3 = __byte_perm(m3, r3, 0x7610);
            // rotate the 8 suffix minima right by r positions inside the lane
            {
                const uint32_t a0 = __funnelshift_l(z3, z0, m.sh16), a1 = __funnelshift_l(z0, z1, m.sh16);
                const uint32_t a2 = __funnelshift_l(z1, z2, m.sh16), a3 = __funnelshift_l(z2, z3, m.sh16);
                z0 = a0; z1 = a1; z2 = a2; z3 = a3;
                if (m.rr & 1) { const uint32_t t = z3; z3 = z2; z2 = z1; z1 = z0; z0 = t; }
                if (m.rr & 2) { uint32_t t = z0; z0 = z2; z2 = t; t = z1; z1 = z3; z3 = t; }
            }
            // fetch: positions >= r come from lane l-q, positions < r from lane l-q-1
            {
                const int dq = m.q, r = m.r;
                uint32_t e0 = shfl_up_inf(z0, dq + (1 < r), lane);
                uint32_t e1 = shfl_up_inf(z1, dq + (3 < r), lane);
                uint32_t e2 = shfl_up_inf(z2, dq + (5 < r), lane);
                uint32_t e3 = shfl_up_inf(z3, dq + (7 < r), lane);
                if (m.jm >= 0) {  // r odd: register jm takes its low half from one lane further down
                    const uint32_t zz = m.jm == 0 ? z0 : (m.jm == 1 ? z1 : (m.jm == 2 ? z2 : z3));
                    const uint32_t x = shfl_up_inf(zz, dq + 1, lane);
                    if (m.jm == 0) e0 = __byte_perm(x, e0, 0x7610);
                    else if (m.jm == 1) e1 = __byte_perm(x, e1, 0x7610);
                    else if (m.jm == 2) e2 = __byte_perm(x, e2, 0x7610);
                    else e3 = __byte_perm(x, e3, 0x7610);
                }
                o0 = vmin2(o0, e0); o1 = vmin2(o1, e1); o2 = vmin2(o2, e2); o3 = vmin2(o3, e3);
            }
            // whole blocks in between: T1 = min B[l-n1 .. l-1], T2 = min B[l-q .. l-1]
            {
                uint32_t T1 = kInf2;
                if (m.n1 >= 1) {
                    uint32_t D = B;  // D = min B[l-2^s+1 .. l] after s doubling steps
                    for (int st = 0; st < m.s; ++st) D = vmin2(D, shfl_up_inf(D, 1 << st, lane));
                    T1 = vmin2(shfl_up_inf(D, 1, lane), shfl_up_inf(D, m.d2, lane));
                }
                const uint32_t T2 = vmin2(T1, shfl_up_inf(B, m.q, lane));
                o0 = vmin2(o0, __byte_perm(T2, T1, m.sel[0]));
                o1 = vmin2(o1, __byte_perm(T2, T1, m.sel[1]));
                o2 = vmin2(o2, __byte_perm(T2, T1, m.sel[2]));
                o3 = vmin2(o3, __byte_perm(T2, T1, m.sel[3]));
            }
            // ---- 3. write the row, offer its last element as a final state ----
            const uint32_t S2 = S | (1u << w);
            if (active)
                *reinterpret_cast<uint4 *>(table_w + ((size_t)S2 * k + w) * Lpad + 8 * lane) =
                    make_uint4(o0, o1, o2, o3);
            if (lane == last_lane) {
                const uint32_t reg = last_reg == 0 ? o0 : (last_reg == 1 ? o1 : (last_reg == 2 ? o2 : o3));
                const uint32_t val = last_half ? (reg >> 16) : (reg & 0xFFFFu);
                if (val != 0xFFFFu) {
                    const unsigned long long key = pack_best(val, level, S2, w);
                    if (key < *reinterpret_cast<volatile unsigned long long *>(d.best)) atomicMin(d.best, key);
                }
            }
        }
    }
}

size_t fast_smem_bytes(const Dev &d)
{
    return (((size_t)d.k * d.k * d.Lpad * 2 + 512 + 15) & ~(size_t)15) + sizeof(WMeta) * PP_MAX_K;
}

template <int NV>
cudaError_t launch_nv(const Dev &d, int level, const FastMeta *meta, unsigned grid, size_t sm, cudaStream_t s)
{
    cudaError_t e = cudaFuncSetAttribute(k_sweep_fast<NV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    k_sweep_fast<NV><<<grid, kFastThreads, sm, s>>>(d, level, meta);
    return cudaGetLastError();
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
        m.q = W >> 3;
        m.r = W & 7;
        m.sh16 = (m.r & 1) ? 16 : 0;
        m.rr = m.r >> 1;
        m.jm = (m.r & 1) ? (m.r >> 1) : -1;
        m.n1 = m.q - 1;
        m.s = 0;
        while (m.n1 >= 1 && (2 << m.s) <= m.n1) ++m.s;
        m.d2 = 1 + m.n1 - (1 << m.s);
        for (int j = 0; j < 4; ++j)
            m.sel[j] = ((2 * j < m.r) ? 0x0010u : 0x0054u) | ((2 * j + 1 < m.r) ? 0x3200u : 0x7600u);
    }
    return true;
}

bool fast_sweep_supported(const Dev &d)
{
    if (d.elem != 2 || d.Lpad > 256 || d.k < 2 || d.k > 19 + 1 || !d.fast_meta) return false;
    int dev = 0, max_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&max_sm, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return false;
    return fast_smem_bytes(d) <= (size_t)max_sm;
}

cudaError_t launch_sweep_fast(const Dev &d, int level, cudaStream_t s)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    unsigned long long n = 1;  // source masks of popcount level-1
    for (int i = 0; i < level - 1; ++i) n = n * (unsigned)(d.k - i) / (unsigned)(i + 1);
    const unsigned wpb = kFastThreads / 32;
    unsigned grid = (unsigned)((n + wpb - 1) / wpb);
    if (grid > (unsigned)sms) grid = (unsigned)sms;
    const size_t sm = fast_smem_bytes(d);
    const FastMeta *meta = static_cast<const FastMeta *>(d.fast_meta);
    switch (level - 1) {
#define PP_CASE(N) case N: return launch_nv<N>(d, level, meta, grid, sm, s);
        PP_CASE(1) PP_CASE(2) PP_CASE(3) PP_CASE(4) PP_CASE(5) PP_CASE(6) PP_CASE(7) PP_CASE(8)
        PP_CASE(9) PP_CASE(10) PP_CASE(11) PP_CASE(12) PP_CASE(13) PP_CASE(14) PP_CASE(15)
        PP_CASE(16) PP_CASE(17) PP_CASE(18) PP_CASE(19)
#undef PP_CASE
    }
    return cudaErrorInvalidValue;
}

}  // namespace pp
