// pp_solve_exact_static: the exact search with every byte of device scratch taken from one
// file-scope array instead of cudaMalloc.  See include/pp.h for the contract.
//
// The array below is linked into the library image, so each GPU that loads libpp holds
// PP_STATIC_SCRATCH_BYTES of device memory until the process exits, used or not.  In host code
// the symbol `g_static_scratch` is only a handle; the device address comes from
// cudaGetSymbolAddress, looked up once per device and cached.
#include <cstring>

#include "pp_internal.cuh"

using namespace pp;

static __device__ __align__(256) unsigned char g_static_scratch[PP_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
constexpr int kStaticMaxK = 14;  // mask list and window table stay on the host stack

unsigned char *g_scratch_addr[kMaxDevices];  // device address of the array, per device ordinal

size_t up256(size_t x) { return (x + 255) / 256 * 256; }

// Device address of the scratch array on the current device (first call per device asks the
// runtime; later calls read the cache).
cudaError_t scratch_address(unsigned char **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = static_cast<unsigned char *>(ptr);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" pp_status pp_solve_exact_static(int32_t L, const uint64_t *layer_out_bits,
                                           const uint64_t *layer_mem_bytes, int32_t k,
                                           const uint64_t *node_mem_bytes, const uint32_t *bw_kbps,
                                           pp_solution *solution_dev, void *cuda_stream)
{
    if (!layer_out_bits || !layer_mem_bytes || !node_mem_bytes || !bw_kbps || !solution_dev)
        return PP_ERR_ARG;
    if (L < 1 || k < 1) return PP_ERR_ARG;
    if (L > PP_MAX_L || k > kStaticMaxK) return PP_ERR_LIMIT;
    for (int i = 0; i < L; ++i)
        if (layer_out_bits[i] >= PP_MAX_BITS) return PP_ERR_LIMIT;
    for (int i = 0; i < k * k; ++i)
        if (bw_kbps[i] >= PP_MAX_KBPS) return PP_ERR_LIMIT;

    // ---- host preparation in fixed-size stack storage (no heap, no device allocation) ----
    uint64_t M[PP_MAX_L + 1];
    M[0] = 0;
    for (int i = 0; i < L; ++i) {
        if (layer_mem_bytes[i] > ~0ull - M[i]) return PP_ERR_LIMIT;
        M[i + 1] = M[i] + layer_mem_bytes[i];
    }
    int16_t pair_u[kStaticMaxK * kStaticMaxK];
    uint32_t ubw[kStaticMaxK * kStaticMaxK];
    int U = 0;
    for (int v = 0; v < k; ++v)
        for (int w = 0; w < k; ++w) {
            uint32_t b = bw_kbps[v * k + w];
            int u = -1;
            if (v != w && b != 0) {
                for (int i = 0; i < U && u < 0; ++i)
                    if (ubw[i] == b) u = i;
                if (u < 0) { u = U; ubw[U++] = b; }
            }
            pair_u[v * k + w] = (int16_t)u;
        }
    if (U == 0) ubw[0] = 0;
    const int elem = ((uint64_t)L * (uint64_t)(U > 0 ? U : 1) + 1 <= 65534) ? 2 : 4;
    const int per32 = 32 / elem;
    const int Lpad = (L + per32 - 1) / per32 * per32;
    const uint32_t nm = 1u << k;

    // scratch layout: small inputs first, then the search tables
    size_t o = 0;
    const size_t o_bits = o;  o = up256(o + (size_t)L * 8);
    const size_t o_M = o;     o = up256(o + (size_t)(L + 1) * 8);
    const size_t o_cap = o;   o = up256(o + (size_t)k * 8);
    const size_t o_bw = o;    o = up256(o + (size_t)k * k * 4);
    const size_t o_lo = o;    o = up256(o + (size_t)k * L * 2);
    const size_t o_pu = o;    o = up256(o + (size_t)k * k * 2);
    const size_t o_ubw = o;   o = up256(o + (size_t)(U > 0 ? U : 1) * 4);
    const size_t o_masks = o; o = up256(o + (size_t)(nm - 1) * 4);
    const size_t o_loff = o;  o = up256(o + (size_t)(k + 2) * 4);
    const size_t o_best = o;  o = up256(o + 8);
    const size_t o_err = o;   o = up256(o + 4);
    const size_t o_pos = o;   o = up256(o + (size_t)L * 2);
    const size_t o_order = o; o = up256(o + (size_t)L * 2);
    const size_t o_gu = o;    o = up256(o + (size_t)(U > 0 ? U : 1) * L * 8);
    const size_t o_cnt = o;   o = up256(o + (size_t)(U > 0 ? U : 1) * L * 4);
    const size_t o_rk = o;    o = up256(o + (size_t)(U > 0 ? U : 1) * L * 4);
    const size_t o_inv = o;   o = up256(o + ((size_t)(U > 0 ? U : 1) * L + 2) * 4);
    const size_t o_rank = o;  o = up256(o + (size_t)k * k * Lpad * elem);
    const size_t o_table = o; o = up256(o + ((size_t)k << k) * Lpad * elem);
    if (o > (size_t)PP_STATIC_SCRATCH_BYTES) return PP_ERR_LIMIT;

    static_assert(kStaticMaxK * PP_MAX_L * 2 <= 64 * 1024, "window table must stay small");
    int16_t lo[kStaticMaxK * PP_MAX_L];
    for (int w = 0; w < k; ++w) {
        int c = 0;
        for (int c2 = 0; c2 < L; ++c2) {
            while (c < c2 && M[c2 + 1] - M[c + 1] > node_mem_bytes[w]) ++c;
            lo[w * L + c2] = (int16_t)c;
        }
    }
    uint32_t level_off[kStaticMaxK + 2];
    uint32_t at[kStaticMaxK + 2];
    static_assert(((1u << kStaticMaxK) - 1) * 4 <= 64 * 1024, "mask list must stay small");
    uint32_t masks[(1u << kStaticMaxK) - 1];
    std::memset(level_off, 0, sizeof level_off);
    for (uint32_t S = 1; S < nm; ++S) level_off[__builtin_popcount(S) + 1]++;
    for (int j = 1; j <= k + 1; ++j) level_off[j] += level_off[j - 1];
    std::memcpy(at, level_off, sizeof at);
    for (uint32_t S = 1; S < nm; ++S) masks[at[__builtin_popcount(S)]++] = S;

    unsigned char *b = nullptr;
    cudaError_t e = scratch_address(&b);
    if (e != cudaSuccess) { cudaGetLastError(); return PP_ERR_CUDA; }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);

    // the sources are pageable host memory: each copy has left the host buffer before it returns
    struct { size_t off; const void *src; size_t bytes; } up[] = {
        {o_bits, layer_out_bits, (size_t)L * 8}, {o_M, M, (size_t)(L + 1) * 8},
        {o_cap, node_mem_bytes, (size_t)k * 8},  {o_bw, bw_kbps, (size_t)k * k * 4},
        {o_lo, lo, (size_t)k * L * 2},           {o_pu, pair_u, (size_t)k * k * 2},
        {o_ubw, ubw, (size_t)(U > 0 ? U : 1) * 4}, {o_masks, masks, (size_t)(nm - 1) * 4},
        {o_loff, level_off, (size_t)(k + 2) * 4}};
    for (auto &q : up) {
        e = cudaMemcpyAsync(b + q.off, q.src, q.bytes, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) { cudaGetLastError(); return PP_ERR_CUDA; }
    }
    // the array keeps whatever the previous call left: reset the words that must start clean
    // (the best-state key and the per-quotient counts are reset by the rank build; every table row
    // is written before it is read)
    e = cudaMemsetAsync(b + o_err, 0, 4, s);
    if (e != cudaSuccess) { cudaGetLastError(); return PP_ERR_CUDA; }

    Dev d{};
    d.L = L; d.k = k; d.Lpad = Lpad; d.U = U; d.elem = elem;
    d.bits = reinterpret_cast<uint64_t *>(b + o_bits);
    d.M = reinterpret_cast<uint64_t *>(b + o_M);
    d.cap = reinterpret_cast<uint64_t *>(b + o_cap);
    d.bw = reinterpret_cast<uint32_t *>(b + o_bw);
    d.lo = reinterpret_cast<int16_t *>(b + o_lo);
    d.pair_u = reinterpret_cast<int16_t *>(b + o_pu);
    d.ubw = reinterpret_cast<uint32_t *>(b + o_ubw);
    d.masks = reinterpret_cast<uint32_t *>(b + o_masks);
    d.level_off = reinterpret_cast<uint32_t *>(b + o_loff);
    d.best = reinterpret_cast<unsigned long long *>(b + o_best);
    d.err = reinterpret_cast<int32_t *>(b + o_err);
    d.pos = reinterpret_cast<int16_t *>(b + o_pos);
    d.order = reinterpret_cast<int16_t *>(b + o_order);
    d.gu = reinterpret_cast<double *>(b + o_gu);
    d.cnt = reinterpret_cast<uint32_t *>(b + o_cnt);
    d.rk = reinterpret_cast<uint32_t *>(b + o_rk);
    d.inv = reinterpret_cast<uint32_t *>(b + o_inv);
    d.rank = b + o_rank;
    d.table = b + o_table;
    d.rank_elems = (uint64_t)k * k * Lpad;
    d.table_elems = ((uint64_t)k << k) * Lpad;

    int launches = 0;
    e = launch_rank_base(d, s, &launches);
    const int top = k < L ? k : L;
    for (int level = 2; level <= top && e == cudaSuccess; ++level) e = launch_sweep_generic(d, level, s);
    if (e == cudaSuccess) e = launch_finalize(d, solution_dev, s, false);
    if (e != cudaSuccess) { cudaGetLastError(); return PP_ERR_CUDA; }
    return PP_OK;
}
